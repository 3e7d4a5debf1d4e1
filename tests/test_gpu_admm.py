"""GPU parity of the ADMM-side primitives (simplex projection, binarisation: Section 5.1; one reduction step of the
library extraction: Algorithm 1) against the CPU oracle, through the C ABI."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import paper_2001_07710_b200 as pc
from paper_2001_07710_b200 import workloads

pytestmark = pytest.mark.gpu


def _all_masks():
    return np.array([sum(1 << b for b in c) for c in itertools.combinations(range(9), 4)], dtype=np.uint16)


def _simplex_tol(d):
    # both sides work in fp64 and round once to fp32; they add in different orders, so a result may land on the
    # neighbouring fp32 value: one unit in the last place of the largest magnitude involved
    return 2.0 ** -23 * max(1.0, float(np.abs(d).max()))


@pytest.mark.parametrize("n,K", [(1, 1), (7, 2), (1000, 4), (1001, 8), (777, 12), (3000, 33), (4099, 126), (513, 256)])
def test_simplex_projection_matches_oracle(n, K):
    rng = np.random.default_rng(n * 1000 + K)
    scale = rng.choice([0.01, 1.0, 25.0], size=(n, 1))
    d = (rng.standard_normal((n, K)) * scale).astype(np.float32)
    d[0] = 0.5                                             # a constant row
    if n > 3:
        d[1] = 0.0; d[1, K // 2] = 9.0                     # one dominant entry: a vertex
        d[2] = np.float32(1.0 / K)                         # already on the simplex (up to rounding)
    u_o, _ = oracle.simplex_project(d)
    buf = torch.full((n * K + 64,), 7.0, dtype=torch.float32, device="cuda")
    u = buf[32:32 + n * K].view(n, K)
    pc.pat_simplex_project(torch.from_numpy(d).cuda(), u)
    torch.cuda.synchronize()
    got = u.cpu().numpy()
    assert np.abs(got - u_o).max() <= _simplex_tol(d)
    assert (got >= 0).all() and np.allclose(got.astype(np.float64).sum(1), 1.0, atol=1e-5)
    assert bool((buf[:32] == 7.0).all()) and bool((buf[32 + n * K:] == 7.0).all())      # nothing outside the output
    assert pc.pat_query_status() == 0


def test_simplex_projection_in_place_and_empty():
    rng = np.random.default_rng(2)
    d = rng.standard_normal((100, 12)).astype(np.float32)
    u_o, _ = oracle.simplex_project(d)
    t = torch.from_numpy(d).cuda()
    pc.pat_simplex_project(t, t)
    assert np.abs(t.cpu().numpy() - u_o).max() <= _simplex_tol(d)
    pc.pat_simplex_project(torch.empty((0, 12), device="cuda"), torch.empty((0, 12), device="cuda"))
    with pytest.raises(pc.PatError):
        pc.pat_simplex_project(torch.zeros((4, 257), device="cuda"))


@pytest.mark.parametrize("n,K", [(1, 1), (9, 2), (1000, 8), (1003, 12), (2500, 126), (300, 256)])
def test_binarisation_matches_oracle(n, K):
    rng = np.random.default_rng(n + K)
    z = rng.standard_normal((n, K)).astype(np.float32)
    z[::3] = np.round(z[::3] * 2) / 2                      # coarse values: many equal maxima, the lowest index must win
    idx_o, hot_o = oracle.argmax_binarize(z)
    idx, hot = pc.pat_argmax_binarize(torch.from_numpy(z).cuda())
    assert np.array_equal(idx.cpu().numpy(), idx_o)        # an index: exact
    assert np.array_equal(hot.cpu().numpy(), hot_o)
    idx2, none = pc.pat_argmax_binarize(torch.from_numpy(z).cuda(), want_onehot=False)
    assert none is None and np.array_equal(idx2.cpu().numpy(), idx_o)


def test_projection_then_binarisation_of_a_selection_variable():
    """The two steps in the order the method takes them: d = z + mu / rho is projected, the result binarised."""
    rng = np.random.default_rng(12)
    n, K = 5000, 8
    z = rng.dirichlet(np.ones(K), size=n)
    d = (z + rng.standard_normal((n, K)) * 0.05).astype(np.float32)
    u = pc.pat_simplex_project(torch.from_numpy(d).cuda())
    idx, _ = pc.pat_argmax_binarize(u, want_onehot=False)
    u_o, _ = oracle.simplex_project(d)
    idx_o, _ = oracle.argmax_binarize(u_o)
    got_u = u.cpu().numpy()
    assert np.abs(got_u - u_o).max() <= _simplex_tol(d)
    # the argmax is decided on each side's own fp32 values: it may differ only where the two largest entries of a
    # row are within the projection's tolerance of each other
    differ = np.nonzero(idx.cpu().numpy() != idx_o)[0]
    for i in differ:
        top = np.sort(u_o[i])[-2:]
        assert top[1] - top[0] <= 2 * _simplex_tol(d)


@pytest.mark.parametrize("shape,K_out", [((64, 64), 12), ((128, 96), 8), ((3, 5), 4), ((256, 256), 12)])
def test_library_extraction_matches_oracle(shape, K_out):
    F, C = shape
    w = workloads.make_weights(np.random.default_rng(F * 7 + C), F, C)
    masks = _all_masks()
    out_o, counts_o = oracle.extract_library(w, masks, K_out)
    out, counts = pc.pat_extract_library(torch.from_numpy(w).cuda(), masks, K_out)
    assert np.array_equal(counts.cpu().numpy(), counts_o)                       # integers: exact
    assert np.array_equal(out.cpu().numpy().view(np.uint16), out_o)
    assert pc.pat_query_status() == 0


def test_library_extraction_schedule_and_ties():
    """126 -> 12 -> 8 -> 4 on the kernels of two layers that share a library; ties and zero kernels."""
    rng = np.random.default_rng(21)
    w = np.concatenate([workloads.make_weights(rng, 64, 64).reshape(-1, 3, 3), workloads.make_weights(rng, 32, 128).reshape(-1, 3, 3)])
    w[::17] = 0.0                                          # all energies equal: mask 0 takes the kernel
    w[5::23] = 0.25                                        # every mask keeps the same energy: lowest id again
    masks_o, masks_g = _all_masks(), _all_masks()
    wg = torch.from_numpy(w).cuda()
    for K_out in (12, 8, 4):
        out_o, counts_o = oracle.extract_library(w, masks_o, K_out)
        out_g, counts_g = pc.pat_extract_library(wg, masks_g, K_out)
        assert np.array_equal(counts_g.cpu().numpy(), counts_o) and int(counts_o.sum()) == len(w)
        masks_g = out_g.cpu().numpy().view(np.uint16).copy()
        assert np.array_equal(masks_g, out_o)
        masks_o = out_o
    # keeping all masks returns the library; the extracted library is accepted by the projection
    same, _ = pc.pat_extract_library(wg, masks_g, 4)
    assert np.array_equal(same.cpu().numpy().view(np.uint16), masks_g)
    pid, _ = pc.pat_project(wg.view(-1, 1, 3, 3)[:4096].reshape(64, 64, 3, 3).contiguous(), masks_g, 512)
    pid_o, _, _ = oracle.project(w[:4096].reshape(64, 64, 3, 3), masks_g, 512)
    assert np.array_equal(pid.cpu().numpy(), pid_o)
    with pytest.raises(pc.PatError):
        pc.pat_extract_library(wg, masks_g, 5)             # more than the library holds


@pytest.mark.parametrize("dtype", ["f16", "f32"])
@pytest.mark.parametrize("shape", [(2, 8, 12, 64), (1, 14, 14, 24), (3, 6, 10, 5), (1, 2, 2, 1), (2, 56, 56, 128)])
@pytest.mark.parametrize("pool", [False, True])
def test_relu_maxpool_matches_oracle(dtype, shape, pool):
    """The rectifier and 2x2 max pooling between layers: the maximum of stored values is exact, so the comparison is too."""
    rng = np.random.default_rng(sum(shape) + pool)
    npdt, tdt = (np.float16, torch.float16) if dtype == "f16" else (np.float32, torch.float32)
    x = rng.standard_normal(shape).astype(npdt)
    ref = oracle.relu_maxpool(x, pool)
    N, H, W, Cc = shape
    n_out = ref.size
    buf = torch.full((n_out + 64,), 7.0, dtype=tdt, device="cuda")
    y = buf[32:32 + n_out].view(ref.shape)
    pc.pat_relu_maxpool(torch.from_numpy(x).cuda(), dtype, pool, y)
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy().astype(np.float64), ref)
    assert bool((buf[:32] == 7.0).all()) and bool((buf[32 + n_out:] == 7.0).all())
    assert pc.pat_query_status() == 0


def test_relu_maxpool_refuses_odd_sizes_and_runs_in_place():
    x = torch.randn((1, 5, 6, 8), device="cuda")
    with pytest.raises(pc.PatError):
        pc.pat_relu_maxpool(x, "f32", True)
    ref = oracle.relu_maxpool(x.cpu().numpy(), False)
    pc.pat_relu_maxpool(x, "f32", False, x)
    assert np.array_equal(x.cpu().numpy().astype(np.float64), ref)

"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import paper_2001_07710_b200 as pc
from paper_2001_07710_b200 import workloads
from helpers import check_close, gpu_project_pack, read_blob, store, stored_weights

pytestmark = pytest.mark.gpu


def _weights(seed, F, C):
    return workloads.make_weights(np.random.default_rng(seed), F, C)


# ------------------------------------------------------------------ projection: bit exact
@pytest.mark.parametrize("F,C,K,num,den", [(8, 8, 8, 3, 10), (64, 64, 8, 3, 10), (37, 53, 12, 1, 8), (128, 64, 4, 1, 4),
                                            (256, 256, 12, 1, 2), (512, 512, 8, 1, 8), (5, 3, 8, 1, 1), (3, 1100, 8, 1, 3)])
def test_project_bit_exact(F, C, K, num, den):
    w = _weights(F * 1000 + C, F, C)
    masks = oracle.library(K)
    n_keep = F * C * num // den
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    pid, wm = pc.pat_project(torch.from_numpy(w).cuda(), pc.pat_library_builtin(K), n_keep)
    assert np.array_equal(pid.cpu().numpy(), pid_o)
    assert np.array_equal(wm.cpu().numpy().view(np.uint32), wm_o.view(np.uint32))


def test_project_full_library_and_in_place():
    masks = np.array([sum(1 << b for b in comb) for comb in itertools.combinations(range(9), 4)], dtype=np.uint16)
    w = _weights(11, 24, 40)
    pid_o, wm_o, _ = oracle.project(w, masks, 300)
    wt = torch.from_numpy(w).cuda()
    pid, wm = pc.pat_project(wt, masks, 300, w_masked=wt)        # w_masked aliases w
    assert wm.data_ptr() == wt.data_ptr()
    assert np.array_equal(pid.cpu().numpy(), pid_o)
    assert np.array_equal(wm.cpu().numpy().view(np.uint32), wm_o.view(np.uint32))


@pytest.mark.parametrize("n_keep", [0, 1, 7, 40, 41, 100, 2047, 2048])
def test_project_ties_and_extremes(n_keep):
    """Many identical kernels (ties at the threshold broken by index), zero kernels, all / none kept."""
    rng = np.random.default_rng(3)
    F, C = 32, 64
    w = np.zeros((F, C, 3, 3), dtype=np.float32)
    base = rng.standard_normal((5, 3, 3)).astype(np.float32)
    choice = rng.integers(0, 6, size=(F, C))
    for i in range(5):
        w[choice == i] = base[i]                                   # choice == 5 stays all-zero
    masks = oracle.library(8)
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    pid, wm = pc.pat_project(torch.from_numpy(w).cuda(), masks, n_keep)
    assert np.array_equal(pid.cpu().numpy(), pid_o)
    assert np.array_equal(wm.cpu().numpy().view(np.uint32), wm_o.view(np.uint32))
    assert int((pid.cpu().numpy() != 255).sum()) == n_keep


@pytest.mark.parametrize("n_keep", [1, 2500, 2731, 5000, 8191])
def test_project_ties_beyond_the_short_list(n_keep):
    """Three distinct kernels over 8192 positions: every threshold has thousands of equal keys, more than the
    selection kernel ranks in shared memory, so its digit-by-digit passes over the candidate list run."""
    rng = np.random.default_rng(11)
    F, C = 64, 128
    base = rng.standard_normal((3, 3, 3)).astype(np.float32)
    w = base[rng.integers(0, 3, size=(F, C))]
    masks = oracle.library(8)
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    pid, wm = pc.pat_project(torch.from_numpy(w).cuda(), masks, n_keep)
    assert np.array_equal(pid.cpu().numpy(), pid_o)
    assert np.array_equal(wm.cpu().numpy().view(np.uint32), wm_o.view(np.uint32))
    assert int((pid.cpu().numpy() != 255).sum()) == n_keep


# ------------------------------------------------------------------ pack: bit exact, round trip
@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("F,C,K,num,den", [(8, 8, 8, 3, 10), (64, 64, 8, 3, 10), (37, 53, 12, 1, 8), (256, 256, 4, 1, 2),
                                            (512, 512, 8, 1, 8), (16, 48, 8, 1, 1), (16, 16, 8, 0, 1)])
def test_pack_bit_exact_and_round_trip(F, C, K, num, den, dtype):
    w = _weights(F * 7 + C, F, C)
    masks = oracle.library(K)
    n_keep = F * C * num // den
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    ref = oracle.pack(wm_o, pid_o, masks, dtype)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, dtype)
    got = read_blob(blob, F, C, K, n_keep, dtype)
    for name in ("perm", "fptr", "pptr", "chan", "w4"):
        assert np.array_equal(got[name], ref[name]), name
    back = pc.pat_unpack(blob, F, C, masks, n_keep, dtype).cpu().numpy()
    if dtype == "f32":
        assert np.array_equal(back.view(np.uint32), wm_o.view(np.uint32))
    else:
        assert np.array_equal(back, wm_o.astype(np.float16).astype(np.float32))
    assert pc.pat_query_status() == 0


def test_blob_mismatch_is_reported_not_executed():
    F, C, K = 16, 16, 8
    masks = oracle.library(K)
    w = _weights(5, F, C)
    pid, wm, blob = gpu_project_pack(w, masks, 64, "f32")
    x = torch.zeros((1, 8, 8, C), device="cuda")
    y = torch.full((1, 8, 8, F), 7.0, device="cuda")
    other = oracle.library(12)[4:12]                                # a different library of the same size
    pc.pat_conv3x3(blob, F, C, other, 64, "f32", x, y=y)
    with pytest.raises(pc.PatError) as e:
        pc.pat_query_status()
    assert e.value.code == 6
    assert float(y.min()) == 7.0                                    # nothing was written
    assert pc.pat_query_status() == 0                               # the word was cleared


# ------------------------------------------------------------------ convolution
CONV_CASES = [
    # N, H, W, C, F, K, keep num/den, stride
    (1, 56, 56, 64, 64, 8, 3, 10, 1),      # config 0
    (2, 20, 37, 24, 40, 8, 1, 4, 1),       # ragged tiles, C and F not multiples of 16/32
    (3, 9, 33, 16, 8, 12, 1, 2, 1),
    (1, 1, 1, 8, 8, 4, 1, 1, 1),           # single pixel
    (2, 14, 14, 128, 96, 8, 1, 8, 1),
    (2, 28, 28, 64, 64, 4, 1, 1, 1),       # nothing pruned by connectivity
    (1, 12, 12, 32, 32, 8, 0, 1, 1),       # everything pruned: output is zero
    (2, 56, 56, 32, 32, 8, 1, 4, 2),       # stride 2, even size
    (2, 15, 23, 16, 24, 12, 1, 2, 2),      # stride 2, odd sizes
    (1, 7, 7, 48, 64, 8, 1, 4, 1),
]


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_matches_oracle(case, dtype):
    N, H, W, C, F, K, num, den, stride = case
    rng = np.random.default_rng(hash(case) % (2 ** 32))
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), dtype)
    masks = oracle.library(K)
    n_keep = F * C * num // den
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    ref = oracle.conv3x3(stored_weights(wm_o, dtype), x, stride)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, dtype)
    y = pc.pat_conv3x3(blob, F, C, masks, n_keep, dtype, torch.from_numpy(x).cuda(), stride)
    assert pc.pat_query_status() == 0
    assert tuple(y.shape) == ref.shape
    check_close(y.float().cpu().numpy(), ref, dtype)
    if n_keep == 0:
        assert not y.any()


# Shapes that take the tuned fp16 kernel (W multiple of 14, even H >= 14, C % 16 == 0, F % 32 == 0): regions that
# straddle two images, images packed side by side (W = 14, 28), batch sizes that leave image slots empty,
# several column groups (W = 112), all three library sizes.
TUNED_CASES = [
    (5, 14, 14, 64, 32, 8, 1, 8),
    (3, 28, 28, 32, 64, 12, 1, 4),
    (3, 56, 56, 32, 32, 8, 1, 8),
    (1, 18, 56, 16, 32, 4, 1, 2),
    (2, 30, 112, 48, 64, 8, 3, 10),
    (1, 224, 224, 16, 32, 8, 1, 8),
    (7, 16, 14, 16, 32, 8, 1, 1),
    (2, 14, 28, 256, 32, 8, 1, 8),
    # more heights for the workspace kernels (4-row thread tiles; a last tile row may be partly outside the image)
    (5, 28, 14, 64, 32, 8, 1, 8),
    (2, 32, 112, 48, 64, 8, 3, 10),
    (3, 44, 28, 32, 32, 4, 1, 2),
    (9, 28, 28, 16, 32, 12, 1, 1),
    (6, 26, 28, 32, 32, 8, 1, 4),
    (9, 13, 14, 32, 64, 8, 1, 4),
]


@pytest.mark.parametrize("use_workspace", [True, False], ids=["workspace", "no_workspace"])
@pytest.mark.parametrize("case", TUNED_CASES)
def test_conv_tuned_f16_matches_oracle(case, use_workspace):
    """Both tuned fp16 kernels: pat_conv3x3_ws (stage images in a workspace) and pat_conv3x3 (no workspace)."""
    N, H, W, C, F, K, num, den = case
    tile_rows = (H + 3) // 4                 # the workspace kernels cover 4 or at least 7 tile rows per image
    assert (pc.pat_conv3x3_workspace(F, C, "f16", N, H, W, 1) > 0) == (tile_rows == 4 or tile_rows >= 7)
    rng = np.random.default_rng(hash(case) % (2 ** 32))
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), "f16")
    masks = oracle.library(K)
    n_keep = F * C * num // den
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    ref = oracle.conv3x3(stored_weights(wm_o, "f16"), x, 1)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, "f16")
    y = torch.full((N, H, W, F), float("nan"), dtype=torch.float16, device="cuda")
    pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", torch.from_numpy(x).cuda(), 1, y=y, use_workspace=use_workspace)
    assert pc.pat_query_status() == 0
    out = y.float().cpu().numpy()
    assert np.isfinite(out).all()                                   # every output element was written
    check_close(out, ref, "f16")


@pytest.mark.parametrize("case", TUNED_CASES)
def test_conv_workspace_f32_matches_oracle(case):
    """The fp32 workspace kernels (stages of 8 channels, 32-byte operations, results written in two rounds) on the
    shapes of the tuned fp16 cases: every output element against the oracle, within the fp32 tolerance."""
    N, H, W, C, F, K, num, den = case
    tile_rows = (H + 3) // 4
    assert (pc.pat_conv3x3_workspace(F, C, "f32", N, H, W, 1) > 0) == (tile_rows == 4 or tile_rows >= 7)
    rng = np.random.default_rng(hash(case) % (2 ** 32) + 1)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), "f32")
    masks = oracle.library(K)
    n_keep = F * C * num // den
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    ref = oracle.conv3x3(stored_weights(wm_o, "f32"), x, 1)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, "f32")
    y = torch.full((N, H, W, F), float("nan"), dtype=torch.float32, device="cuda")
    pc.pat_conv3x3(blob, F, C, masks, n_keep, "f32", torch.from_numpy(x).cuda(), 1, y=y)
    assert pc.pat_query_status() == 0
    out = y.cpu().numpy()
    assert np.isfinite(out).all()                                   # every output element was written
    check_close(out, ref, "f32")


def test_conv_workspace_f32_cut_items_and_arbitrary_library():
    """fp32 workspace kernels with a remainder of work items (pieces + reduce kernel) and with masks outside the
    built-in set (position-by-position code); sampled against the oracle, and against the generic kernel."""
    N, H, W, C, F = 24, 56, 56, 32, 128
    masks = np.array([0b000001111, 0b111100000, 0b101000101, 0x03A, 0x0D8, 0b100110001], dtype=np.uint16)
    rng = np.random.default_rng(78)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), "f32")
    n_keep = F * C // 4
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, "f32")
    xt = torch.from_numpy(x).cuda()
    y = torch.full((N, H, W, F), float("nan"), dtype=torch.float32, device="cuda")
    pc.pat_conv3x3(blob, F, C, masks, n_keep, "f32", xt, 1, y=y)
    assert pc.pat_query_status() == 0
    assert bool(torch.isfinite(y).all())
    coords = np.stack([rng.integers(0, N, 6000), rng.integers(0, H, 6000), rng.integers(0, W, 6000), rng.integers(0, F, 6000)], axis=1).astype(np.int32)
    coords[:2000, 0] = rng.integers(20, 24, 2000)          # the last images belong to the cut items
    ref = oracle.conv3x3_at(stored_weights(wm_o, "f32"), x, coords, 1)
    out = y[coords[:, 0], coords[:, 1], coords[:, 2], coords[:, 3]].cpu().numpy()
    check_close(out, ref, "f32")
    y2 = pc.pat_conv3x3(blob, F, C, masks, n_keep, "f32", xt, 1, use_workspace=False)
    assert torch.allclose(y, y2, rtol=1e-4, atol=1e-5)


@pytest.mark.parametrize("dtype", ["f16", "f32"])
@pytest.mark.parametrize("case", [(9, 7, 7, 32, 64, 8, 1, 4), (5, 12, 10, 16, 32, 12, 1, 2), (3, 3, 14, 32, 32, 8, 1, 1), (6, 16, 5, 16, 32, 4, 1, 2)])
def test_conv_workspace_small_images(case, dtype):
    """Images smaller than a thread tile (fewer than 14 columns) or than four tile rows (fewer than 13 rows) take a
    whole tile column / four tile rows of the workspace kernels; the pixels outside the image are neither read nor written."""
    N, H, W, C, F, K, num, den = case
    assert pc.pat_conv3x3_workspace(F, C, dtype, N, H, W, 1) > 0
    rng = np.random.default_rng(hash(case) % (2 ** 32) + 7)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), dtype)
    masks = oracle.library(K)
    n_keep = F * C * num // den
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    ref = oracle.conv3x3(stored_weights(wm_o, dtype), x, 1)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, dtype)
    tdt = torch.float16 if dtype == "f16" else torch.float32
    # the output sits inside a larger buffer filled with a marker: nothing outside it may be written
    buf = torch.full((N * H * W * F + 4096,), 7.0, dtype=tdt, device="cuda")
    y = buf[2048:2048 + N * H * W * F].view(N, H, W, F)
    y.fill_(float("nan"))
    pc.pat_conv3x3(blob, F, C, masks, n_keep, dtype, torch.from_numpy(x).cuda(), 1, y=y)
    assert pc.pat_query_status() == 0
    out = y.float().cpu().numpy()
    assert np.isfinite(out).all()
    check_close(out, ref, dtype)
    assert bool((buf[:2048] == 7.0).all()) and bool((buf[2048 + N * H * W * F:] == 7.0).all())


@pytest.mark.parametrize("dtype", ["f16", "f32"])
@pytest.mark.parametrize("case", [(3, 56, 56, 32, 64, 8, 1, 4), (5, 14, 14, 64, 32, 8, 1, 2), (2, 28, 28, 16, 32, 12, 1, 1), (4, 7, 7, 32, 32, 8, 1, 4),
                                  (24, 28, 56, 64, 64, 8, 1, 8)])
def test_conv_workspace_stride2(case, dtype):
    """Stride 2 on the workspace kernels (computed like stride 1; the results at even rows and columns are written),
    odd and even sizes, cut items included: every output element against the oracle."""
    N, H, W, C, F, K, num, den = case
    assert pc.pat_conv3x3_workspace(F, C, dtype, N, H, W, 2) > 0
    rng = np.random.default_rng(hash(case) % (2 ** 32) + 11)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), dtype)
    masks = oracle.library(K)
    n_keep = F * C * num // den
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    ref = oracle.conv3x3(stored_weights(wm_o, dtype), x, 2)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, dtype)
    y = pc.pat_conv3x3(blob, F, C, masks, n_keep, dtype, torch.from_numpy(x).cuda(), 2)
    assert pc.pat_query_status() == 0
    assert tuple(y.shape) == ref.shape
    out = y.float().cpu().numpy()
    assert np.isfinite(out).all()
    check_close(out, ref, dtype)


def test_conv_workspace_entry_point_agrees_with_plain_entry_point():
    """pat_conv3x3_ws and pat_conv3x3 add the kernels of a filter in different orders: fp16 results agree to a
    rounding step; a caller-owned workspace full of NaN bit patterns is overwritten before it is read."""
    N, H, W, C, F, K = 6, 28, 28, 128, 96, 8
    rng = np.random.default_rng(5)
    w = workloads.make_weights(rng, F, C)
    xt = torch.from_numpy(store(workloads.make_inputs(rng, N, H, W, C), "f16")).cuda()
    masks = oracle.library(K)
    n_keep = F * C // 8
    _, _, blob = gpu_project_pack(w, masks, n_keep, "f16")
    ws = torch.full((pc.pat_conv3x3_workspace(F, C, "f16", N, H, W, 1),), 0xFF, dtype=torch.uint8, device="cuda")
    y0 = pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", xt, 1, use_workspace=False)
    y1 = pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", xt, 1, workspace=ws)
    assert pc.pat_query_status() == 0
    assert bool(torch.isfinite(y1).all())
    assert torch.allclose(y0.float(), y1.float(), rtol=2e-3, atol=2e-4)


def test_conv_workspace_cut_items():
    """More work items than SMs with a remainder: the items of the last round are cut along the input channels,
    run as pieces on different blocks and are added up by the reduce kernel; sampled against the oracle."""
    N, H, W, C, F, K = 24, 56, 56, 64, 128, 8
    rng = np.random.default_rng(77)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), "f16")
    masks = oracle.library(K)
    n_keep = F * C // 8
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, "f16")
    y = torch.full((N, H, W, F), float("nan"), dtype=torch.float16, device="cuda")
    pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", torch.from_numpy(x).cuda(), 1, y=y)
    assert pc.pat_query_status() == 0
    assert bool(torch.isfinite(y).all())
    coords = np.stack([rng.integers(0, N, 8000), rng.integers(0, H, 8000), rng.integers(0, W, 8000), rng.integers(0, F, 8000)], axis=1).astype(np.int32)
    coords[:2000, 0] = rng.integers(20, 24, 2000)          # the last images belong to the cut items
    ref = oracle.conv3x3_at(stored_weights(wm_o, "f16"), x, coords, 1)
    out = y[coords[:, 0], coords[:, 1], coords[:, 2], coords[:, 3]].float().cpu().numpy()
    check_close(out, ref, "f16")
    y2 = pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", torch.from_numpy(x).cuda(), 1, use_workspace=False)
    assert torch.allclose(y.float(), y2.float(), rtol=2e-3, atol=2e-4)


@pytest.mark.parametrize("use_workspace", [True, False], ids=["workspace", "no_workspace"])
def test_conv_tuned_f16_many_regions_dense_keep(use_workspace):
    """Several work items per thread block (672 regions) and up to 16 kernels per filter and 16-channel block
    (keep 1/2, 12 patterns; descriptor blocks too large for the five-slot ring); sampled against the oracle."""
    N, H, W, C, F, K = 12, 224, 224, 16, 128, 12
    rng = np.random.default_rng(99)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), "f16")
    masks = oracle.library(K)
    n_keep = F * C // 2
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, "f16")
    y = torch.full((N, H, W, F), float("nan"), dtype=torch.float16, device="cuda")
    pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", torch.from_numpy(x).cuda(), 1, y=y, use_workspace=use_workspace)
    assert pc.pat_query_status() == 0
    assert bool(torch.isfinite(y).all())
    coords = np.stack([rng.integers(0, N, 6000), rng.integers(0, H, 6000), rng.integers(0, W, 6000), rng.integers(0, F, 6000)], axis=1).astype(np.int32)
    coords[:64, 1] = 0; coords[64:128, 1] = H - 1; coords[128:192, 2] = 0; coords[192:256, 2] = W - 1
    ref = oracle.conv3x3_at(stored_weights(wm_o, "f16"), x, coords, 1)
    out = y[coords[:, 0], coords[:, 1], coords[:, 2], coords[:, 3]].float().cpu().numpy()
    check_close(out, ref, "f16")


def test_conv_tuned_f16_arbitrary_library():
    """Masks outside the built-in set (some without the centre) run through the per-position code of the tuned kernel."""
    N, H, W, C, F = 3, 28, 28, 48, 64
    masks = np.array([0b000001111, 0b111100000, 0b101000101, 0b010101010 & 0x1FF | 0, 0x03A, 0x0D8, 0b100110001], dtype=np.uint16)
    masks = np.array([m for m in masks if bin(int(m)).count("1") == 4], dtype=np.uint16)
    assert len(masks) >= 6
    rng = np.random.default_rng(77)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), "f16")
    n_keep = F * C // 4
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    ref = oracle.conv3x3(stored_weights(wm_o, "f16"), x, 1)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, "f16")
    assert np.array_equal(pid.cpu().numpy(), pid_o)
    y = pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", torch.from_numpy(x).cuda(), 1)
    assert pc.pat_query_status() == 0
    check_close(y.float().cpu().numpy(), ref, "f16")


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("N,H,W,C,F,stride", [(2, 40, 70, 3, 64, 1), (1, 9, 9, 1, 8, 1), (2, 17, 33, 3, 40, 2), (1, 16, 16, 16, 32, 1),
                                             (2, 10, 37, 3, 64, 1), (1, 8, 32, 3, 64, 1), (3, 5, 64, 3, 64, 1)])
def test_dense_conv_matches_oracle(N, H, W, C, F, stride, dtype):
    rng = np.random.default_rng(N * 1000 + H)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), dtype)
    ref = oracle.conv3x3(stored_weights(w, dtype), x, stride)
    y = pc.pat_conv3x3_dense(torch.from_numpy(w).cuda(), dtype, torch.from_numpy(x).cuda(), stride)
    check_close(y.float().cpu().numpy(), ref, dtype)


# ------------------------------------------------------------------ refused inputs and failed waits
def test_pack_refuses_wrong_n_keep_and_writes_nothing_outside_the_blob():
    """pattern_id keeps more kernels than the n_keep given to pat_pack: the blob is refused (status PAT_ERR_BLOB,
    magic cleared) and no kernel writes past the sections sized by n_keep: the blob sits inside a buffer of
    canary bytes that must stay untouched."""
    F, C, K = 64, 64, 8
    masks = oracle.library(K)
    w = torch.from_numpy(_weights(11, F, C)).cuda()
    pid, wm = pc.pat_project(w, masks, F * C // 2)                   # 2048 kernels kept
    for dtype in ("f32", "f16"):
        n_wrong = F * C // 8                                         # pack is told 512
        size = pc.pat_pack_size(F, C, K, n_wrong, dtype)
        pad = 1 << 20
        buf = torch.full((size + 2 * pad,), 0xC5, dtype=torch.uint8, device="cuda")
        blob = buf[pad:pad + size]
        assert blob.data_ptr() % 256 == 0
        pc.pat_pack(wm, pid, masks, n_wrong, dtype, blob=blob)
        with pytest.raises(pc.PatError) as e:
            pc.pat_query_status()
        assert e.value.code == 6
        assert bool((buf[:pad] == 0xC5).all()) and bool((buf[pad + size:] == 0xC5).all())
        assert int(blob[:4].view(torch.int32)[0]) == 0               # the header's magic: the blob cannot be used
    assert pc.pat_query_status() == 0


@pytest.mark.parametrize("dtype", ["f16", "f32"])
def test_blob_mismatch_on_the_workspace_path_writes_nothing(dtype):
    """A blob packed with another library, on a shape the workspace kernels cover with cut items (one small image:
    the reduce kernel would run): the status word says PAT_ERR_BLOB and y is untouched; the same holds for a header
    whose magic or version word was overwritten."""
    N, H, W, C, F, K = 1, 28, 28, 64, 32, 8
    masks = oracle.library(K)
    n_keep = F * C // 4
    _, _, blob = gpu_project_pack(_weights(12, F, C), masks, n_keep, dtype)
    tdt = torch.float16 if dtype == "f16" else torch.float32
    x = torch.zeros((N, H, W, C), dtype=tdt, device="cuda")
    assert pc.pat_conv3x3_workspace(F, C, dtype, N, H, W, 1) > 0
    other = oracle.library(12)[4:12]

    def refused(blob_, masks_):
        y = torch.full((N, H, W, F), 7.0, dtype=tdt, device="cuda")
        pc.pat_conv3x3(blob_, F, C, masks_, n_keep, dtype, x, 1, y=y)
        with pytest.raises(pc.PatError) as e:
            pc.pat_query_status()
        assert e.value.code == 6
        assert float(y.min()) == 7.0 and float(y.max()) == 7.0

    refused(blob, other)
    for word in (0, 1):                                              # magic, version
        bad = blob.clone()
        bad[4 * word:4 * word + 4] = 0x5A
        refused(bad, masks)
    assert pc.pat_query_status() == 0
    y = pc.pat_conv3x3(blob, F, C, masks, n_keep, dtype, x, 1)        # the intact blob still runs
    assert pc.pat_query_status() == 0 and not y.any()


def test_bounded_wait_runs_out_and_is_reported():
    """The copies of one pipeline stage are never issued (test hook) and the wait limit is 1 ms: the kernel must
    end by itself, report PAT_ERR_TIMEOUT once, and leave the device usable: the next, normal call matches the
    oracle."""
    N, H, W, C, F, K = 4, 56, 56, 64, 64, 8
    rng = np.random.default_rng(31)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), "f16")
    masks = oracle.library(K)
    n_keep = F * C // 8
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    _, _, blob = gpu_project_pack(w, masks, n_keep, "f16")
    xt = torch.from_numpy(x).cuda()
    assert pc.pat_conv3x3_workspace(F, C, "f16", N, H, W, 1) > 0
    try:
        pc.pat_debug_set(0, 1_000_000)       # 1 ms
        pc.pat_debug_set(1, 1)               # second stage of every thread block
        pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", xt, 1)
        with pytest.raises(pc.PatError) as e:
            pc.pat_query_status()
        assert e.value.code == 9
    finally:
        pc.pat_debug_set(1, -1)
        pc.pat_debug_set(0, 0)
    assert pc.pat_query_status() == 0        # the word was cleared
    y = pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", xt, 1)
    assert pc.pat_query_status() == 0
    check_close(y.float().cpu().numpy(), oracle.conv3x3(stored_weights(wm_o, "f16"), x, 1), "f16")


@pytest.mark.parametrize("dtype", ["f16", "f32"])
@pytest.mark.parametrize("case", [(3, 56, 56, 32, 64, 8, 1, 4, 1), (5, 14, 14, 64, 32, 8, 1, 2, 1), (2, 28, 28, 16, 32, 12, 1, 1, 2),
                                  (24, 28, 56, 64, 64, 8, 1, 8, 1), (1, 28, 28, 64, 64, 8, 1, 8, 1), (2, 23, 17, 24, 40, 8, 1, 2, 1)])
def test_conv_with_fused_rectifier(case, dtype):
    """pat_conv3x3_ws_act: max(conv, 0) written by the convolution's own epilogue (whole items, cut items whose sums
    pass through the reduce kernel, a small batch that is cut entirely, stride 2, and a shape the workspace kernels do
    not cover: convolution, then the rectifier in place) - every element against the oracle's relu(conv)."""
    N, H, W, C, F, K, num, den, stride = case
    rng = np.random.default_rng(hash(case) % (2 ** 32) + 5)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), dtype)
    masks = oracle.library(K)
    n_keep = F * C * num // den
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    ref = np.maximum(oracle.conv3x3(stored_weights(wm_o, dtype), x, stride), 0.0)
    assert (ref == 0).mean() > 0.2                      # the rectifier has something to do
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, dtype)
    y = pc.pat_conv3x3(blob, F, C, masks, n_keep, dtype, torch.from_numpy(x).cuda(), stride, relu=True)
    assert pc.pat_query_status() == 0
    out = y.float().cpu().numpy()
    assert tuple(out.shape) == ref.shape and (out >= 0).all()
    check_close(out, ref, dtype)
    # where the reference is clearly negative before the rectifier the output is exactly zero
    pre = oracle.conv3x3(stored_weights(wm_o, dtype), x, stride)
    assert (out[pre < -1e-2] == 0).all()


@pytest.mark.parametrize("dtype", ["f16", "f32"])
@pytest.mark.parametrize("case", [(3, 56, 56, 32, 64, 8, 1, 4), (5, 14, 14, 64, 32, 8, 1, 2), (24, 28, 56, 64, 64, 8, 1, 8),
                                  (1, 28, 28, 64, 64, 8, 1, 8), (9, 8, 8, 16, 32, 12, 1, 1), (2, 30, 28, 32, 32, 4, 1, 2)])
def test_conv_with_fused_rectifier_and_pooling(case, dtype):
    """pat_conv3x3_ws_act(act = 2): the pooled image max(0, 2 x 2 block of conv) written by the convolution's own
    epilogue (whole items, cut items through the pooling reduce kernel, a batch that is cut entirely, 14 x 14 images
    whose last tile row is half empty, images narrower than a thread tile, a height that is no multiple of 4) -
    every element against the oracle's relu_maxpool(conv), and bit for bit against the two-pass result of the
    library itself (same sums, monotone rounding)."""
    N, H, W, C, F, K, num, den = case
    rng = np.random.default_rng(hash(case) % (2 ** 32) + 11)
    w = workloads.make_weights(rng, F, C)
    x = store(workloads.make_inputs(rng, N, H, W, C), dtype)
    masks = oracle.library(K)
    n_keep = F * C * num // den
    pid_o, wm_o, _ = oracle.project(w, masks, n_keep)
    ref = oracle.relu_maxpool(oracle.conv3x3(stored_weights(wm_o, dtype), x, 1), True)
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, dtype)
    xt = torch.from_numpy(x).cuda()
    assert pc.pat_conv3x3_workspace(F, C, dtype, N, H, W, 1) > 0
    y = torch.full((N, H // 2, W // 2, F), float("nan"), dtype=xt.dtype, device="cuda")
    pc.pat_conv3x3(blob, F, C, masks, n_keep, dtype, xt, 1, y=y, pool=True)
    assert pc.pat_query_status() == 0
    out = y.float().cpu().numpy()
    assert tuple(out.shape) == ref.shape and np.isfinite(out).all() and (out >= 0).all()
    check_close(out, ref, dtype)
    two_pass = pc.pat_relu_maxpool(pc.pat_conv3x3(blob, F, C, masks, n_keep, dtype, xt, 1), dtype, True)
    assert torch.equal(two_pass, y)


def test_fused_pooling_refuses_what_it_cannot_pool():
    """act = 2 with stride 2, an odd height, or a layer without workspace kernels: PAT_ERR_SHAPE, nothing written."""
    F, C, K = 32, 16, 8
    masks = oracle.library(K)
    w = _weights(9, F, C)
    n_keep = F * C // 2
    pid, wm, blob = gpu_project_pack(w, masks, n_keep, "f16")
    for (N, H, W, stride) in [(1, 28, 28, 2), (1, 15, 14, 1), (1, 24, 46, 1)]:
        x = torch.zeros((N, H, W, C), dtype=torch.float16, device="cuda")
        y = torch.full((N, H // 2, W // 2, F), 7.0, dtype=torch.float16, device="cuda")
        with pytest.raises(pc.PatError) as e:
            pc.pat_conv3x3(blob, F, C, masks, n_keep, "f16", x, stride, y=y, pool=True)
        assert e.value.code == 2                                        # PAT_ERR_SHAPE
        torch.cuda.synchronize()
        assert float(y.min()) == 7.0
    assert pc.pat_query_status() == 0

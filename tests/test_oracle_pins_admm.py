"""Pins of the oracle's ADMM-side primitives: simplex projection and binarisation (Section 5.1) and one reduction
step of the library extraction (Algorithm 1, Section 5.2).  CPU only; nothing here touches the CUDA library."""
import itertools

import numpy as np
import pytest

import oracle


def _all_masks():
    return np.array([sum(1 << b for b in c) for c in itertools.combinations(range(9), 4)], dtype=np.uint16)


# ----------------------------------------------------------------------------------------- simplex projection
def _root_by_bisection(d):
    """nu with sum(max(d - nu, 0)) = 1, found on the defining equation itself (float64 bisection)."""
    d = d.astype(np.float64)
    lo, hi = d.max() - 1.0, d.max()          # g(lo) >= 1 >= g(hi) = 0
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if np.maximum(d - mid, 0.0).sum() > 1.0:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


@pytest.mark.parametrize("K", [1, 2, 3, 8, 12, 126])
def test_simplex_root_solves_the_defining_equation(K):
    rng = np.random.default_rng(K)
    d = np.concatenate([rng.standard_normal((40, K)) * s for s in (0.01, 1.0, 30.0)]).astype(np.float32)
    u, nu = oracle.simplex_project(d)
    for i in range(len(d)):
        ref = _root_by_bisection(d[i])
        assert abs(nu[i] - ref) <= 1e-12 * max(1.0, abs(ref))
        expect = np.maximum(d[i].astype(np.float64) - ref, 0.0)
        assert np.allclose(u[i], expect, rtol=0, atol=1e-6 * max(1.0, np.abs(d[i]).max()))


def test_simplex_optimality_conditions():
    rng = np.random.default_rng(5)
    d = (rng.standard_normal((200, 12)) * 2).astype(np.float32)
    u, nu = oracle.simplex_project(d)
    u64, d64 = u.astype(np.float64), d.astype(np.float64)
    assert (u64 >= 0).all()
    assert np.allclose(u64.sum(1), 1.0, atol=1e-6)
    for i in range(len(d)):
        on = u64[i] > 0
        # on the support d - u is the same number (the multiplier), off the support d is not above it
        assert np.allclose(d64[i][on] - u64[i][on], nu[i], atol=1e-6)
        assert (d64[i][~on] <= nu[i] + 1e-12).all()
    # the projection is the closest point: no random point of the simplex is closer
    for i in range(20):
        p = rng.dirichlet(np.ones(12), size=200)
        assert (np.square(p - d64[i]).sum(1) >= np.square(u64[i] - d64[i]).sum() - 1e-9).all()


def test_simplex_closed_forms():
    rng = np.random.default_rng(6)
    # a point of the simplex is its own projection
    p = rng.dirichlet(np.ones(8), size=50).astype(np.float32)
    u, nu = oracle.simplex_project(p)
    assert np.allclose(u, p, atol=2e-7) and np.allclose(nu, (p.astype(np.float64).sum(1) - 1) / 8, atol=1e-7)
    # a constant vector goes to the centre, whatever the constant
    for c in (-7.5, 0.0, 3.25):
        u, _ = oracle.simplex_project(np.full((1, 5), c, dtype=np.float32))
        assert np.allclose(u, 0.2, atol=1e-7)
    # one entry ahead of all others by at least 1: a vertex
    d = np.array([[0.3, 2.0, 0.9, -1.0]], dtype=np.float32)
    u, nu = oracle.simplex_project(d)
    assert np.array_equal(u, np.array([[0, 1, 0, 0]], dtype=np.float32)) and nu[0] == 1.0
    # K = 1: always 1.  K = 2: u = clip((1 + d0 - d1) / 2, 0, 1)
    u, _ = oracle.simplex_project(np.array([[-4.0], [9.0]], dtype=np.float32))
    assert np.array_equal(u, np.ones((2, 1), dtype=np.float32))
    d2 = (rng.standard_normal((100, 2)) * 1.5).astype(np.float32)
    u, _ = oracle.simplex_project(d2)
    u0 = np.clip((1.0 + d2[:, 0].astype(np.float64) - d2[:, 1]) / 2, 0, 1)
    assert np.allclose(u[:, 0], u0, atol=2e-7) and np.allclose(u[:, 1], 1 - u0, atol=2e-7)
    # adding a constant to every entry changes nothing; the worked example (0.5, 0.8, -0.1) -> nu = 0.15
    d = rng.standard_normal((30, 9)).astype(np.float32)
    ua, _ = oracle.simplex_project(d)
    ub, _ = oracle.simplex_project((d.astype(np.float64) + 2.0).astype(np.float32))
    assert np.allclose(ua, ub, atol=1e-6)
    u, nu = oracle.simplex_project(np.array([[0.5, 0.8, -0.1]], dtype=np.float32))
    assert np.allclose(nu, 0.15, atol=1e-7) and np.allclose(u, [[0.35, 0.65, 0.0]], atol=1e-7)


def test_binarisation_is_the_closest_one_hot_vector():
    rng = np.random.default_rng(7)
    z = rng.standard_normal((300, 12)).astype(np.float32)
    idx, onehot = oracle.argmax_binarize(z)
    assert np.array_equal(idx, np.argmax(z, axis=1))
    eye = np.eye(12)
    for i in range(len(z)):
        dist = np.square(eye - z[i].astype(np.float64)).sum(1)        # distance to every admissible vector
        assert dist[idx[i]] == dist.min()
        assert np.array_equal(onehot[i], eye[idx[i]].astype(np.float32))
    # equal maxima: the lowest index (the declared convention)
    idx, _ = oracle.argmax_binarize(np.array([[1, 3, 3, 0], [2, 2, 2, 2]], dtype=np.float32))
    assert list(idx) == [1, 0]


# ----------------------------------------------------------------------------------------- library extraction
def test_extraction_counts_equal_top4_magnitude_histogram():
    """With all C(9,4) masks the best mask of a kernel holds its four largest magnitudes (no ties in random data)."""
    rng = np.random.default_rng(8)
    w = rng.standard_normal((5000, 3, 3)).astype(np.float32)
    masks = _all_masks()
    out, counts = oracle.extract_library(w, masks, 12)
    top4 = np.argsort(-np.abs(w.reshape(-1, 9)), axis=1)[:, :4]
    bits = (1 << top4).sum(1)
    where = {int(m): j for j, m in enumerate(masks)}
    ref = np.zeros(126, dtype=np.int64)
    for b in bits:
        ref[where[int(b)]] += 1
    assert np.array_equal(counts, ref) and counts.sum() == 5000
    order = sorted(range(126), key=lambda j: (-ref[j], j))[:12]
    assert list(out) == [int(masks[j]) for j in sorted(order)]


def test_extraction_recovers_planted_patterns():
    rng = np.random.default_rng(9)
    masks = _all_masks()
    planted = [17, 80, 5, 111, 64, 33]                     # ids in the full library
    freq = [400, 300, 200, 100, 50, 25]
    ws = []
    for j, f in zip(planted, freq):
        k = rng.uniform(-0.1, 0.1, size=(f, 9)).astype(np.float32)
        for b in range(9):
            if masks[j] >> b & 1:
                k[:, b] = rng.choice([-1.0, 1.0], size=f) * rng.uniform(1.0, 2.0, size=f)
        ws.append(k)
    w = np.concatenate(ws)
    w = w[rng.permutation(len(w))]                         # the order of the kernels does not matter
    out, counts = oracle.extract_library(w, masks, 4)
    assert [int(counts[j]) for j in planted] == freq and counts.sum() == sum(freq)
    assert [int(m) for m in out] == [int(masks[j]) for j in sorted(planted[:4])]   # survivors keep the library's order
    # a second step on the reduced library: every kernel is re-assigned inside it
    out2, counts2 = oracle.extract_library(w, out, 2)
    assert counts2.sum() == sum(freq) and len(out2) == 2
    assert set(int(m) for m in out2) == {int(masks[17]), int(masks[80])}
    # keeping everything is the identity; scaling the weights changes nothing
    same, _ = oracle.extract_library(w, masks, 126)
    assert np.array_equal(same, masks)
    out3, counts3 = oracle.extract_library(w * 3.0, masks, 4)
    assert np.array_equal(out3, out) and np.array_equal(counts3, counts)


def test_extraction_tie_rules():
    masks = oracle.library(8)
    # all-zero kernels: every energy is 0, the lowest id takes them all; equal counts: lower ids stay
    out, counts = oracle.extract_library(np.zeros((10, 3, 3), dtype=np.float32), masks, 3)
    assert counts[0] == 10 and counts[1:].sum() == 0
    assert list(out) == [int(m) for m in masks[:3]]


# ----------------------------------------------------------------------------------------- rectifier and pooling
def test_relu_maxpool_matches_library_ops():
    import torch
    rng = np.random.default_rng(10)
    x = rng.standard_normal((2, 6, 8, 5))
    t = torch.from_numpy(x).permute(0, 3, 1, 2)
    relu = torch.relu(t)
    assert np.array_equal(oracle.relu_maxpool(x, False), relu.permute(0, 2, 3, 1).numpy())
    pooled = torch.nn.functional.max_pool2d(relu, 2, 2).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(oracle.relu_maxpool(x, True), pooled)
    # by hand: one channel, one 2x2 block; all negative -> 0
    assert oracle.relu_maxpool(np.array([[[[-1.0], [3.0]], [[2.0], [-5.0]]]]), True).tolist() == [[[[3.0]]]]
    assert oracle.relu_maxpool(np.array([[[[-1.0], [-3.0]], [[-2.0], [-5.0]]]]), True).tolist() == [[[[0.0]]]]
    with pytest.raises(ValueError):
        oracle.relu_maxpool(np.zeros((1, 3, 4, 1)), True)

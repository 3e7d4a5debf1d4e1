"""Pins of the CPU oracle against what the paper and the mathematics fix (CPU only)."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "library_family_sums.txt")


def _gold():
    out = {}
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        out[k] = [int(t) for t in v]
    return out


def _mask_matrix(m):
    return np.array([(int(m) >> b) & 1 for b in range(9)]).reshape(3, 3)


def _all_masks():
    return np.array([sum(1 << b for b in comb) for comb in itertools.combinations(range(9), 4)], dtype=np.uint16)


# ------------------------------------------------------------------ pattern library (Section 4.2, 5.1)
def test_library_family_sums_match_paper():
    g = _gold()
    lib = oracle.library(12)
    cross = sum(_mask_matrix(m) for m in lib[0:4])
    block = sum(_mask_matrix(m) for m in lib[4:8])
    assert cross.ravel().tolist() == g["cross_family_sum"]
    assert block.ravel().tolist() == g["block_family_sum"]
    # every arm of the cross family appears in 3 of 4 masks: p = 0.75
    assert cross[0, 1] / 4 == 0.75


def test_library_basic_properties():
    for K in (4, 8, 12):
        lib = oracle.library(K)
        assert len(set(lib.tolist())) == K
        for m in lib:
            assert bin(int(m)).count("1") == 4          # four entries per kernel (Section 5.1)
            assert int(m) & (1 << 4)                    # centre always kept
    # nested libraries: 4 subset of 8 subset of 12
    assert oracle.library(12)[:8].tolist() == oracle.library(8).tolist()
    assert oracle.library(8)[:4].tolist() == oracle.library(4).tolist()
    with pytest.raises(ValueError):
        oracle.library(5)


def test_library_families_closed_under_rotation():
    def rot(m):
        out = 0
        for b in range(9):
            if m & (1 << b):
                r, s = divmod(b, 3)
                out |= 1 << (3 * s + (2 - r))
        return out
    lib = oracle.library(12).tolist()
    for fam in (lib[0:4], lib[4:8], lib[8:12]):
        assert sorted(rot(m) for m in fam) == sorted(fam)


def test_full_library_size_and_compression():
    g = _gold()
    assert len(_all_masks()) == g["full_library_size"][0]
    assert 9 * 100 // 4 == g["pattern_compression_x100"][0]


# ------------------------------------------------------------------ projection
def test_project_full_library_equals_top4_magnitudes():
    """With all 126 masks the best pattern keeps the 4 largest |w| (textbook top-k)."""
    rng = np.random.default_rng(1)
    w = rng.standard_normal((6, 7, 3, 3)).astype(np.float32)
    masks = _all_masks()
    pid, wm, g2 = oracle.project(w, masks, 6 * 7)
    flat = w.reshape(-1, 9)
    for i, k in enumerate(flat):
        top4 = np.argsort(-np.abs(k.astype(np.float64)), kind="stable")[:4]
        expect = np.zeros(9, dtype=np.float32)
        expect[top4] = k[top4]
        assert np.array_equal(wm.reshape(-1, 9)[i], expect)
        assert int(masks[pid.ravel()[i]]) == sum(1 << int(b) for b in top4)
        assert g2.ravel()[i] >= 4.0 / 9.0 * float((k.astype(np.float64) ** 2).sum()) - 1e-15


def test_project_kernel_that_is_a_scaled_mask_selects_it():
    lib = oracle.library(8)
    w = np.zeros((1, 8, 3, 3), dtype=np.float32)
    for j, m in enumerate(lib):
        w[0, j] = (_mask_matrix(m) * (j + 1.5)).astype(np.float32)
    pid, wm, g2 = oracle.project(w, lib, 8)
    assert pid.ravel().tolist() == list(range(8))
    assert np.array_equal(wm, w)                               # 100 % of the energy retained
    assert np.allclose(g2.ravel(), [4 * (j + 1.5) ** 2 for j in range(8)])


def test_project_hand_case_and_tie_breaks():
    lib = oracle.library(8)
    # all-equal kernel: every mask keeps the same energy -> lowest id (0) wins
    w = np.ones((1, 2, 3, 3), dtype=np.float32)
    # second kernel: energy only in the bottom-right 2x2 block -> id 7
    w[0, 1] = 0
    w[0, 1, 1:, 1:] = [[1, 2], [3, 4]]
    pid, wm, g2 = oracle.project(w, lib, 2)
    assert pid.ravel().tolist() == [0, 7]
    assert g2.ravel().tolist() == [4.0, 30.0]
    # connectivity ties: identical kernels -> lower linear index is kept
    w2 = np.ones((2, 2, 3, 3), dtype=np.float32)
    pid2, wm2, _ = oracle.project(w2, lib, 3)
    assert pid2.ravel().tolist() == [0, 0, 0, 255]
    assert not wm2[1, 1].any()


@pytest.mark.parametrize("K", [4, 8, 12])
def test_project_invariants(K):
    rng = np.random.default_rng(K)
    F, Cc = 12, 10
    w = rng.standard_normal((F, Cc, 3, 3)).astype(np.float32)
    lib = oracle.library(K)
    n_keep = (F * Cc * 3) // 10
    pid, wm, g2 = oracle.project(w, lib, n_keep)
    kept = pid != 255
    assert kept.sum() == n_keep
    # chosen energy is maximal over the library (brute force, independent arithmetic in numpy)
    sq = w.astype(np.float64) ** 2
    for f in range(F):
        for c in range(Cc):
            e = [sum(sq[f, c].ravel()[b] for b in range(9) if (int(m) >> b) & 1) for m in lib]
            assert g2[f, c] == max(e)
            assert g2[f, c] <= sq[f, c].sum() + 1e-15
            if kept[f, c]:
                assert e[pid[f, c]] == max(e) and pid[f, c] == int(np.argmax(e))
                mm = _mask_matrix(lib[pid[f, c]]).astype(bool)
                assert np.array_equal(wm[f, c][mm], w[f, c][mm])         # kept bits identical
                assert not wm[f, c][~mm].any()                           # everything else zero
                assert not np.signbit(wm[f, c][~mm]).any()               # and +0.0
            else:
                assert not wm[f, c].any() and not np.signbit(wm[f, c]).any()
    # connectivity: every kept kernel is at least as strong as every removed one (Section 6.1)
    assert g2[kept].min() >= g2[~kept].max()
    # compression identity: overall = 2.25 / keep ratio
    assert abs(9 * F * Cc / (4 * n_keep) - 2.25 / (n_keep / (F * Cc))) < 1e-12


def test_project_extremes_and_filter_permutation():
    rng = np.random.default_rng(5)
    w = rng.standard_normal((5, 6, 3, 3)).astype(np.float32)
    lib = oracle.library(8)
    pid_all, wm_all, _ = oracle.project(w, lib, 30)
    assert (pid_all != 255).all()
    pid_none, wm_none, _ = oracle.project(w, lib, 0)
    assert (pid_none == 255).all() and not wm_none.any()
    perm = rng.permutation(5)
    pid, wm, _ = oracle.project(w, lib, 11)
    pid_p, wm_p, _ = oracle.project(w[perm], lib, 11)
    assert np.array_equal(pid_p, pid[perm]) and np.array_equal(wm_p, wm[perm])


# ------------------------------------------------------------------ fp16 rounding
def test_f16_rounding_matches_ieee_library_conversion():
    rng = np.random.default_rng(2)
    vals = np.concatenate([
        rng.standard_normal(3000).astype(np.float32),
        (rng.standard_normal(2000) * 1e-5).astype(np.float32),         # subnormal halves
        (rng.standard_normal(500) * 7e4).astype(np.float32),           # overflow to inf
        np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 6e-8, 2.98e-8, 2.9802322e-8, 2.99e-8,
                  1.0 + 2 ** -11, 1.0 + 2 ** -11 + 2 ** -20, 1.0 + 3 * 2 ** -11, np.inf, -np.inf], dtype=np.float32)])
    got = oracle.f32_to_f16_bits(vals)
    with np.errstate(over="ignore"):
        ref = vals.astype(np.float16).view(np.uint16)
    assert np.array_equal(got, ref)


def test_f16_exhaustive_round_trip():
    L = oracle.lib()
    bits = np.arange(65536, dtype=np.uint16)
    as_f32 = bits.view(np.float16).astype(np.float32)
    finite = np.isfinite(as_f32)
    back = oracle.f32_to_f16_bits(as_f32[finite])
    assert np.array_equal(back, bits[finite])
    for b in (0x0001, 0x03FF, 0x0400, 0x3C00, 0x7BFF, 0xC000):
        assert L.orc_f16_to_f64(b) == float(np.uint16(b).view(np.float16))


# ------------------------------------------------------------------ pack
@pytest.mark.parametrize("dtype", ["f32", "f16"])
def test_pack_invariants_and_round_trip(dtype):
    rng = np.random.default_rng(7)
    F, Cc, K = 20, 24, 8
    lib = oracle.library(K)
    w = rng.standard_normal((F, Cc, 3, 3)).astype(np.float32)
    pid, wm, _ = oracle.project(w, lib, F * Cc // 4)
    pk = oracle.pack(wm, pid, lib, dtype)
    perm, fptr, pptr, chan, w4 = pk["perm"], pk["fptr"], pk["pptr"], pk["chan"], pk["w4"]
    assert sorted(perm.tolist()) == list(range(F))
    assert fptr[0] == 0 and fptr[F] == F * Cc // 4 and (np.diff(fptr) >= 0).all()
    counts = np.diff(fptr)
    assert (np.diff(counts) <= 0).all()                       # kept counts non-increasing
    assert np.array_equal(counts, (pid[perm] != 255).sum(axis=1))
    # ordering key: (count desc, histogram desc lexicographic, index asc)
    keys = [(-int(counts[q]),) + tuple(-int((pid[perm[q]] == j).sum()) for j in range(K)) + (int(perm[q]),) for q in range(F)]
    assert keys == sorted(keys)
    # round trip to dense masked weights
    dense = np.zeros_like(wm)
    for q in range(F):
        assert pptr[q, 0] == fptr[q] and pptr[q, K] == fptr[q + 1]
        for j in range(K):
            seg = chan[pptr[q, j]:pptr[q, j + 1]]
            assert (np.diff(seg.astype(int)) > 0).all()        # channels strictly ascending
            bits = [b for b in range(9) if (int(lib[j]) >> b) & 1]
            for k in range(pptr[q, j], pptr[q, j + 1]):
                assert pid[perm[q], chan[k]] == j
                for t, b in enumerate(bits):
                    if dtype == "f32":
                        dense[perm[q], chan[k]].reshape(9)[b] = w4[k, t].view(np.float32)
                    else:
                        dense[perm[q], chan[k]].reshape(9)[b] = np.uint16(w4[k, t]).view(np.float16)
    if dtype == "f32":
        assert np.array_equal(dense.view(np.uint32), wm.view(np.uint32))
    else:
        assert np.array_equal(dense, wm.astype(np.float16).astype(np.float32))


# ------------------------------------------------------------------ convolution
def _torch_conv(wm, x, stride):
    xt = torch.from_numpy(np.ascontiguousarray(x.astype(np.float64).transpose(0, 3, 1, 2)))
    wt = torch.from_numpy(wm.astype(np.float64))
    return torch.nn.functional.conv2d(xt, wt, stride=stride, padding=1).numpy().transpose(0, 2, 3, 1)


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("shape", [(2, 7, 9, 5, 6), (1, 8, 8, 3, 4), (1, 1, 1, 2, 3), (1, 2, 5, 4, 2)])
def test_conv_matches_library_conv2d(shape, stride):
    N, H, W, Cc, F = shape
    rng = np.random.default_rng(H * 100 + W)
    x = rng.standard_normal((N, H, W, Cc)).astype(np.float32)
    w = rng.standard_normal((F, Cc, 3, 3)).astype(np.float32)
    y = oracle.conv3x3(w, x, stride)
    ref = _torch_conv(w, x, stride)
    assert y.shape == ref.shape
    assert np.abs(y - ref).max() <= 1e-12 * (1 + np.abs(ref).max())


def test_conv_delta_input_reads_kernel_reversed():
    """A unit impulse at (2,2) puts w[f,c,r,s] at output (2+1-r, 2+1-s): correlation, not convolution."""
    Cc, F = 3, 2
    w = np.arange(F * Cc * 9, dtype=np.float32).reshape(F, Cc, 3, 3) + 1
    for c in range(Cc):
        x = np.zeros((1, 5, 5, Cc), dtype=np.float32)
        x[0, 2, 2, c] = 1.0
        y = oracle.conv3x3(w, x)
        for f in range(F):
            assert np.array_equal(y[0, 1:4, 1:4, f], w[f, c, ::-1, ::-1].astype(np.float64))
            assert y[0, :, :, f].sum() == w[f, c].sum()


def test_conv_identity_kernel_and_padding():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((2, 6, 4, 3)).astype(np.float32)
    w = np.zeros((3, 3, 3, 3), dtype=np.float32)
    for c in range(3):
        w[c, c, 1, 1] = 1.0
    assert np.array_equal(oracle.conv3x3(w, x), x.astype(np.float64))
    # all-ones input, single-tap kernels: the tap at (r,s) reads outside the image on one border
    ones = np.ones((1, 4, 5, 1), dtype=np.float32)
    for r in range(3):
        for s in range(3):
            k = np.zeros((1, 1, 3, 3), dtype=np.float32)
            k[0, 0, r, s] = 1.0
            y = oracle.conv3x3(k, ones)[0, :, :, 0]
            expect = np.ones((4, 5))
            if r == 0: expect[0, :] = 0
            if r == 2: expect[-1, :] = 0
            if s == 0: expect[:, 0] = 0
            if s == 2: expect[:, -1] = 0
            assert np.array_equal(y, expect)


def test_conv_stride2_is_subsampled_stride1_and_linear():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 9, 8, 4)).astype(np.float32)
    x2 = rng.standard_normal((2, 9, 8, 4)).astype(np.float32)
    w = rng.standard_normal((5, 4, 3, 3)).astype(np.float32)
    y1 = oracle.conv3x3(w, x, 1)
    y2 = oracle.conv3x3(w, x, 2)
    assert np.array_equal(y2, y1[:, ::2, ::2, :])
    ysum = oracle.conv3x3(w, (x.astype(np.float64) + 2 * x2.astype(np.float64)), 1)
    assert np.abs(ysum - (y1 + 2 * oracle.conv3x3(w, x2, 1))).max() < 1e-12
    yw = oracle.conv3x3(3 * w.astype(np.float64), x, 1)
    assert np.abs(yw - 3 * y1).max() < 1e-12


def test_conv_of_masked_weights_equals_independent_sparse_gather():
    """Sparse definition (only stored taps, gathered by channel) == dense conv of masked weights."""
    rng = np.random.default_rng(6)
    N, H, W, Cc, F = 2, 6, 7, 8, 9
    lib = oracle.library(8)
    w = rng.standard_normal((F, Cc, 3, 3)).astype(np.float32)
    x = np.maximum(rng.standard_normal((N, H, W, Cc)), 0).astype(np.float32)
    pid, wm, _ = oracle.project(w, lib, F * Cc * 3 // 10)
    for stride in (1, 2):
        y = oracle.conv3x3(wm, x, stride)
        Ho, Wo = y.shape[1:3]
        xp = np.zeros((N, H + 2, W + 2, Cc))
        xp[:, 1:-1, 1:-1] = x
        ref = np.zeros_like(y)
        for f in range(F):
            for c in range(Cc):
                if pid[f, c] == 255:
                    continue
                for b in range(9):
                    if (int(lib[pid[f, c]]) >> b) & 1:
                        r, s = divmod(b, 3)
                        ref[..., f] += float(w[f, c, r, s]) * xp[:, r:r + stride * Ho:stride, s:s + stride * Wo:stride, c]
        assert np.abs(y - ref).max() <= 1e-12 * (1 + np.abs(ref).max())
        # sampled evaluation agrees with the full one
        coords = np.array([[n, yy, xx, f] for n in range(N) for yy in (0, Ho - 1) for xx in (0, Wo // 2) for f in (0, F - 1)], dtype=np.int32)
        pts = oracle.conv3x3_at(wm, x, coords, stride)
        assert np.array_equal(pts, y[coords[:, 0], coords[:, 1], coords[:, 2], coords[:, 3]])


def test_conv_accepts_f16_storage():
    rng = np.random.default_rng(8)
    x = np.maximum(rng.standard_normal((1, 5, 5, 4)), 0).astype(np.float16)
    w = rng.standard_normal((3, 4, 3, 3)).astype(np.float16)
    y = oracle.conv3x3(w.astype(np.float64), x)
    ref = _torch_conv(w.astype(np.float64), x.astype(np.float64), 1)
    assert np.abs(y - ref).max() < 1e-12

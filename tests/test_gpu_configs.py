"""Full-size parity on the five evaluation configurations, in the launch configuration bench.py times.

Projection and packing are compared bit for bit with the oracle on every layer.  The convolution output of the
full batch is compared element by element on whole images - the first, the middle and the last of the batch - for
every layer whose single image costs the oracle's direct float64 definition at most WHOLE_IMAGE_MACS multiply-adds
(test id "...-whole"; all layers of the five configurations do), and on sampled coordinates of all images (all
corners and edges of the first and last image plus seeded random points); a layer above that cost would be
compared on the samples only (id "...-sampled").  Every output element is also checked to have been written
(finite) and the status word to be clean.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2001_07710_b200 as pc
from paper_2001_07710_b200 import workloads
from helpers import check_close, read_blob

pytestmark = pytest.mark.gpu

N_RANDOM = 3000
POOLED_LAYERS = ("conv2", "conv4", "conv7", "conv10", "conv13")   # Section 7's VGG-16: pooling after these
WHOLE_IMAGE_MACS = 2.5e9      # dense 9 * C * F * Ho * Wo of one image: about a second of the oracle on 16 cores


def _whole(L) -> bool:
    return 9.0 * L.C * L.F * L.Ho * L.Wo <= WHOLE_IMAGE_MACS


def _sample_coords(rng, N, Ho, Wo, F):
    pts = []
    for n in {0, N - 1}:
        for y in {0, 1, Ho // 2, Ho - 2 if Ho > 1 else 0, Ho - 1}:
            for x in {0, 1, Wo // 2, Wo - 2 if Wo > 1 else 0, Wo - 1}:
                for f in {0, F // 2, F - 1}:
                    pts.append((n, max(y, 0), max(x, 0), f))
    rnd = np.stack([rng.integers(0, N, N_RANDOM), rng.integers(0, Ho, N_RANDOM),
                    rng.integers(0, Wo, N_RANDOM), rng.integers(0, F, N_RANDOM)], axis=1)
    return np.concatenate([np.array(pts, dtype=np.int64), rnd]).astype(np.int32)


def _check_layer(cfg, L):
    dtype = cfg.dtype
    w, x = workloads.make_layer_tensors(cfg.number, L, cfg.N)
    xs = x.astype(np.float16) if dtype == "f16" else x
    del x
    xt = torch.from_numpy(xs).cuda()
    rng = np.random.default_rng(workloads.layer_seed(cfg.number, L) + 1)
    coords = _sample_coords(rng, cfg.N, L.Ho, L.Wo, L.F)
    if L.dense:
        wst = w.astype(np.float16).astype(np.float64) if dtype == "f16" else w.astype(np.float64)
        y = pc.pat_conv3x3_dense(torch.from_numpy(w).cuda(), dtype, xt, L.stride)
    else:
        masks = oracle.library(L.K)
        assert np.array_equal(masks, pc.pat_library_builtin(L.K))
        pid_o, wm_o, _ = oracle.project(w, masks, L.n_keep)
        pid, wm = pc.pat_project(torch.from_numpy(w).cuda(), masks, L.n_keep)
        assert np.array_equal(pid.cpu().numpy(), pid_o)
        assert np.array_equal(wm.cpu().numpy().view(np.uint32), wm_o.view(np.uint32))
        blob = pc.pat_pack(wm, pid, masks, L.n_keep, dtype)
        ref_pack = oracle.pack(wm_o, pid_o, masks, dtype)
        got = read_blob(blob, L.F, L.C, L.K, L.n_keep, dtype)
        for name in ("perm", "fptr", "pptr", "chan", "w4"):
            assert np.array_equal(got[name], ref_pack[name]), name
        wst = wm_o.astype(np.float16).astype(np.float64) if dtype == "f16" else wm_o.astype(np.float64)
        y = pc.pat_conv3x3(blob, L.F, L.C, masks, L.n_keep, dtype, xt, L.stride)
    assert pc.pat_query_status() == 0
    assert tuple(y.shape) == (cfg.N, L.Ho, L.Wo, L.F)
    assert bool(torch.isfinite(y).all())
    ref = oracle.conv3x3_at(wst, xs, coords, L.stride)
    out = y[coords[:, 0], coords[:, 1], coords[:, 2], coords[:, 3]].float().cpu().numpy()
    check_close(out, ref, dtype)
    # the layers of the VGG-16 stack that 2x2 max pooling follows: the pooled image written by the convolution's own
    # epilogue equals, bit for bit and over the whole batch, the pooling pass run on the full-size output
    pooled = None
    if not L.dense and cfg.number in (1, 3) and L.name in POOLED_LAYERS:
        pooled = pc.pat_conv3x3(blob, L.F, L.C, masks, L.n_keep, dtype, xt, L.stride, pool=True)
        assert pc.pat_query_status() == 0
        assert torch.equal(pooled, pc.pat_relu_maxpool(y, dtype, True))
    if _whole(L):
        for n in sorted({0, cfg.N // 2, cfg.N - 1}):
            ref_img = oracle.conv3x3(wst, xs[n:n + 1], L.stride)
            check_close(y[n:n + 1].float().cpu().numpy(), ref_img, dtype)
            if pooled is not None:
                check_close(pooled[n:n + 1].float().cpu().numpy(), oracle.relu_maxpool(ref_img, True), dtype)


def _layers(cfg_no):
    cfg = workloads.configs()[cfg_no]
    return [pytest.param(cfg_no, i, id=f"cfg{cfg_no}-{L.name}-{'whole' if _whole(L) else 'sampled'}")
            for i, L in enumerate(cfg.layers)]


@pytest.mark.parametrize("cfg_no,layer_idx", _layers(0) + _layers(1) + _layers(2) + _layers(3) + _layers(4))
def test_config_layer(cfg_no, layer_idx):
    cfg = workloads.configs()[cfg_no]
    _check_layer(cfg, cfg.layers[layer_idx])
    torch.cuda.empty_cache()

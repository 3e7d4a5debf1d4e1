"""Shared test helpers: run the CUDA pipeline through the binding, run the oracle, compare."""
import numpy as np
import torch

import oracle
import paper_2001_07710_b200 as pc

FP32_TOL = 1e-4          # |err| <= 1e-4 * (1 + |ref|)
FP16_REL, FP16_ABS = 2e-2, 1e-4   # |err| <= 2e-2 * |ref| + 1e-4


def gpu_project_pack(w_np, masks, n_keep, dtype):
    w = torch.from_numpy(w_np).cuda()
    pid, wm = pc.pat_project(w, masks, n_keep)
    blob = pc.pat_pack(wm, pid, masks, n_keep, dtype)
    return pid, wm, blob


def read_blob(blob, F, C, K, n_keep, dtype):
    """Canonical arrays of a blob as numpy arrays (w4 as bit patterns)."""
    raw = blob.cpu().numpy()
    off = pc.pat_blob_layout(F, C, K, n_keep, dtype)
    e = 2 if dtype == "f16" else 4
    perm = raw[off["perm"]:off["perm"] + 4 * F].view(np.int32)
    fptr = raw[off["fptr"]:off["fptr"] + 4 * (F + 1)].view(np.int32)
    pptr = raw[off["pptr"]:off["pptr"] + 4 * F * (K + 1)].view(np.int32).reshape(F, K + 1)
    chan = raw[off["chan"]:off["chan"] + 2 * n_keep].view(np.uint16)
    w4 = raw[off["w4"]:off["w4"] + 4 * e * n_keep].view(np.uint16 if e == 2 else np.uint32).reshape(n_keep, 4)
    return dict(perm=perm, fptr=fptr, pptr=pptr, chan=chan, w4=w4.astype(np.uint32))


def store(x_np, dtype):
    """Round fp32 activations to the storage type (fp16: round to nearest even, numpy's conversion)."""
    return x_np.astype(np.float16) if dtype == "f16" else x_np


def stored_weights(wm_np, dtype):
    """Masked weights as the blob stores them, widened to float64."""
    if dtype == "f16":
        return wm_np.astype(np.float16).astype(np.float64)
    return wm_np.astype(np.float64)


def check_close(out, ref, dtype):
    out = np.asarray(out, dtype=np.float64)
    err = np.abs(out - ref)
    if dtype == "f16":
        bound = FP16_REL * np.abs(ref) + FP16_ABS
    else:
        bound = FP32_TOL * (1.0 + np.abs(ref))
    bad = err > bound
    assert not bad.any(), f"{bad.sum()} of {bad.size} outside tolerance; worst err {err.max():.3e} (ref {ref.ravel()[err.argmax()]:.3e})"
    return float(err.max())

"""CPU oracle for pattern-based sparse 3x3 convolution.  TEST INFRASTRUCTURE ONLY.

Thin ctypes front end of ``patoracle.c`` (plain C, float64, OpenMP).  It shares no code with the
CUDA library and must only be used by the tests, the smoke check and the CPU-baseline leg of the
benchmark.  All arithmetic lives in the C file; this module marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "patoracle.c")
_LIB = os.path.join(_HERE, "libpatoracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_library.argtypes = [C.c_int, C.c_void_p]
        L.orc_project.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int64,
                                  C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_f32_to_f16.argtypes = [C.c_float]
        L.orc_f32_to_f16.restype = C.c_uint16
        L.orc_f16_to_f64.argtypes = [C.c_uint16]
        L.orc_f16_to_f64.restype = C.c_double
        L.orc_pack.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int,
                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_conv3x3.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                  C.c_int, C.c_void_p]
        L.orc_conv3x3_at.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                     C.c_int, C.c_void_p, C.c_int64, C.c_void_p]
        L.orc_simplex_project.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_argmax_binarize.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_extract_library.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_relu_maxpool.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p]
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def library(K: int) -> np.ndarray:
    """The built-in pattern library of size 4, 8 or 12 as 9-bit masks (bit 3*r+s)."""
    m = np.zeros(K, dtype=np.uint16)
    if lib().orc_library(K, _p(m)) != 0:
        raise ValueError("library size must be 4, 8 or 12")
    return m


def project(w: np.ndarray, masks: np.ndarray, n_keep: int):
    """Pattern selection + connectivity pruning.  Returns (pid u8 [F,C], w_masked f32, gamma2 f64)."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    F, Cc = w.shape[:2]
    masks = np.ascontiguousarray(masks, dtype=np.uint16)
    pid = np.empty((F, Cc), dtype=np.uint8)
    wm = np.empty_like(w)
    g2 = np.empty((F, Cc), dtype=np.float64)
    rc = lib().orc_project(_p(w), F, Cc, _p(masks), len(masks), int(n_keep), _p(pid), _p(wm), _p(g2))
    if rc != 0:
        raise ValueError(f"orc_project failed ({rc})")
    return pid, wm, g2


def f32_to_f16_bits(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint16)
    f = lib().orc_f32_to_f16
    flat_in, flat_out = a.ravel(), out.ravel()
    for i in range(flat_in.size):
        flat_out[i] = f(float(flat_in[i]))
    return out


def pack(wm: np.ndarray, pid: np.ndarray, masks: np.ndarray, dtype: str = "f32"):
    """Canonical pack.  Returns dict(perm, fptr, pptr, chan, w4); w4 holds bit patterns (u32)."""
    wm = np.ascontiguousarray(wm, dtype=np.float32)
    pid = np.ascontiguousarray(pid, dtype=np.uint8)
    masks = np.ascontiguousarray(masks, dtype=np.uint16)
    F, Cc = pid.shape
    K = len(masks)
    n_keep = int((pid != 0xFF).sum())
    perm = np.empty(F, dtype=np.int32)
    fptr = np.empty(F + 1, dtype=np.int32)
    pptr = np.empty((F, K + 1), dtype=np.int32)
    chan = np.empty(n_keep, dtype=np.uint16)
    w4 = np.empty((n_keep, 4), dtype=np.uint32)
    rc = lib().orc_pack(_p(wm), _p(pid), F, Cc, _p(masks), K, {"f32": 0, "f16": 1}[dtype],
                        _p(perm), _p(fptr), _p(pptr), _p(chan), _p(w4))
    if rc != 0:
        raise ValueError(f"orc_pack failed ({rc})")
    return dict(perm=perm, fptr=fptr, pptr=pptr, chan=chan, w4=w4)


def _act(x: np.ndarray):
    if x.dtype == np.float64:
        return np.ascontiguousarray(x), 0
    if x.dtype == np.float32:
        return np.ascontiguousarray(x), 1
    if x.dtype == np.float16:
        return np.ascontiguousarray(x).view(np.uint16), 2
    raise TypeError("activations must be float64, float32 or float16")


def conv3x3(wm: np.ndarray, x: np.ndarray, stride: int = 1) -> np.ndarray:
    """Direct dense float64 cross-correlation of (masked) weights [F,C,3,3] with NHWC x, pad 1."""
    wm = np.ascontiguousarray(wm, dtype=np.float64)
    F, Cc = wm.shape[:2]
    xa, dt = _act(x)
    N, H, W, Cx = x.shape
    assert Cx == Cc
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    y = np.empty((N, Ho, Wo, F), dtype=np.float64)
    rc = lib().orc_conv3x3(_p(wm), F, Cc, _p(xa), dt, N, H, W, stride, _p(y))
    if rc != 0:
        raise ValueError(f"orc_conv3x3 failed ({rc})")
    return y


def conv3x3_at(wm: np.ndarray, x: np.ndarray, coords: np.ndarray, stride: int = 1) -> np.ndarray:
    """The same definition at listed output coordinates (rows of (n, y, x, f))."""
    wm = np.ascontiguousarray(wm, dtype=np.float64)
    F, Cc = wm.shape[:2]
    xa, dt = _act(x)
    N, H, W, Cx = x.shape
    assert Cx == Cc
    coords = np.ascontiguousarray(coords, dtype=np.int32)
    out = np.empty(len(coords), dtype=np.float64)
    rc = lib().orc_conv3x3_at(_p(wm), F, Cc, _p(xa), dt, N, H, W, stride, _p(coords), len(coords), _p(out))
    if rc != 0:
        raise ValueError(f"orc_conv3x3_at failed ({rc})")
    return out


def simplex_project(d: np.ndarray):
    """Projection of every row of d [n,K] (fp32) onto the probability simplex.  Returns (u f32 [n,K], nu f64 [n])."""
    d = np.ascontiguousarray(d, dtype=np.float32)
    n, K = d.shape
    u = np.empty_like(d)
    nu = np.empty(n, dtype=np.float64)
    rc = lib().orc_simplex_project(_p(d), n, K, _p(u), _p(nu))
    if rc != 0:
        raise ValueError(f"orc_simplex_project failed ({rc})")
    return u, nu


def argmax_binarize(z: np.ndarray):
    """Index of the largest entry of every row of z [n,K] (lowest index on ties) and the one-hot rows."""
    z = np.ascontiguousarray(z, dtype=np.float32)
    n, K = z.shape
    idx = np.empty(n, dtype=np.uint8)
    onehot = np.empty_like(z)
    rc = lib().orc_argmax_binarize(_p(z), n, K, _p(idx), _p(onehot))
    if rc != 0:
        raise ValueError(f"orc_argmax_binarize failed ({rc})")
    return idx, onehot


def extract_library(w: np.ndarray, masks: np.ndarray, K_out: int):
    """One reduction step of the library extraction on kernels w [n,3,3].  Returns (masks_out u16 [K_out], counts i64 [K_in])."""
    w = np.ascontiguousarray(w, dtype=np.float32).reshape(-1, 9)
    masks = np.ascontiguousarray(masks, dtype=np.uint16)
    out = np.empty(K_out, dtype=np.uint16)
    counts = np.empty(len(masks), dtype=np.int64)
    rc = lib().orc_extract_library(_p(w), len(w), _p(masks), len(masks), int(K_out), _p(out), _p(counts))
    if rc != 0:
        raise ValueError(f"orc_extract_library failed ({rc})")
    return out, counts


def relu_maxpool(x: np.ndarray, pool: bool) -> np.ndarray:
    """max(x, 0) and, if pool, 2x2 max pooling with stride 2, on NHWC x (any float dtype; computed in float64)."""
    x64 = np.ascontiguousarray(x, dtype=np.float64)
    N, H, W, Cc = x64.shape
    y = np.empty((N, H // 2, W // 2, Cc) if pool else (N, H, W, Cc), dtype=np.float64)
    rc = lib().orc_relu_maxpool(_p(x64), N, H, W, Cc, 1 if pool else 0, _p(y))
    if rc != 0:
        raise ValueError(f"orc_relu_maxpool failed ({rc})")
    return y

"""ctypes binding of libpatconv.so: same names as the C ABI, argument marshalling only.

PyTorch is used for device memory and streams.  Every computation runs in the CUDA library; there is no
fallback: loading fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libpatconv.so")

PAT_F32, PAT_F16 = 0, 1
PAT_PRUNED = 0xFF
_DT = {"f32": PAT_F32, "f16": PAT_F16, PAT_F32: PAT_F32, PAT_F16: PAT_F16,
       torch.float32: PAT_F32, torch.float16: PAT_F16}
TORCH_DTYPE = {PAT_F32: torch.float32, PAT_F16: torch.float16}

EXPORTS = ["pat_strerror", "pat_last_error", "pat_library_builtin", "pat_project_workspace", "pat_project",
           "pat_pack_size", "pat_pack", "pat_blob_layout", "pat_unpack", "pat_conv3x3", "pat_conv3x3_dense",
           "pat_query_status", "pat_launch_count", "pat_project_static", "pat_project_static_max_kernels",
           "pat_conv3x3_workspace", "pat_conv3x3_ws", "pat_debug_set", "pat_measure_fma_peak",
           "pat_simplex_project", "pat_argmax_binarize", "pat_extract_library", "pat_relu_maxpool", "pat_conv3x3_ws_act"]


class PatError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"patconv error {code}: {message}")
        self.code = code


_lib = None


def load() -> C.CDLL:
    """Load the CUDA library (raises if it has not been built: there is no other code path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2001_07710_b200.build` (nvcc, sm_100a)")
    L = C.CDLL(_LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int, C.c_int64, C.c_size_t
    L.pat_strerror.argtypes = [i32]; L.pat_strerror.restype = C.c_char_p
    L.pat_last_error.argtypes = []; L.pat_last_error.restype = C.c_char_p
    L.pat_library_builtin.argtypes = [i32, vp]
    L.pat_project_workspace.argtypes = [i32, i32]; L.pat_project_workspace.restype = sz
    L.pat_project.argtypes = [vp, i32, i32, vp, i32, i64, vp, vp, vp, sz, vp]
    L.pat_pack_size.argtypes = [i32, i32, i32, i64, i32]; L.pat_pack_size.restype = sz
    L.pat_pack.argtypes = [vp, vp, i32, i32, vp, i32, i64, i32, vp, sz, vp]
    L.pat_blob_layout.argtypes = [i32, i32, i32, i64, i32, vp]
    L.pat_unpack.argtypes = [vp, i32, i32, vp, i32, i64, i32, vp, vp]
    L.pat_conv3x3.argtypes = [vp, i32, i32, vp, i32, i64, i32, vp, vp, i32, i32, i32, i32, vp]
    L.pat_conv3x3_workspace.argtypes = [i32, i32, i32, i32, i32, i32, i32]; L.pat_conv3x3_workspace.restype = sz
    L.pat_conv3x3_ws.argtypes = [vp, i32, i32, vp, i32, i64, i32, vp, vp, i32, i32, i32, i32, vp, sz, vp]
    L.pat_conv3x3_dense.argtypes = [vp, i32, i32, i32, vp, vp, i32, i32, i32, i32, vp]
    L.pat_query_status.argtypes = [vp]
    L.pat_launch_count.argtypes = []; L.pat_launch_count.restype = C.c_uint64
    L.pat_project_static.argtypes = [vp, i32, i32, vp, i32, i64, vp, vp, vp]
    L.pat_project_static_max_kernels.argtypes = []; L.pat_project_static_max_kernels.restype = i64
    L.pat_debug_set.argtypes = [i32, C.c_longlong]
    L.pat_measure_fma_peak.argtypes = [i32, vp, sz, vp, vp]
    L.pat_simplex_project.argtypes = [vp, i64, i32, vp, vp]
    L.pat_argmax_binarize.argtypes = [vp, i64, i32, vp, vp, vp]
    L.pat_extract_library.argtypes = [vp, i64, vp, i32, i32, vp, vp, vp]
    L.pat_relu_maxpool.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp, vp]
    L.pat_conv3x3_ws_act.argtypes = [vp, i32, i32, vp, i32, i64, i32, vp, vp, i32, i32, i32, i32, i32, vp, sz, vp]
    _lib = L
    return L


def _check(rc: int):
    if rc != 0:
        raise PatError(rc, load().pat_last_error().decode())


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _masks(masks: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(masks, dtype=np.uint16))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def pat_library_builtin(K: int) -> np.ndarray:
    m = np.zeros(max(K, 1), dtype=np.uint16)
    _check(load().pat_library_builtin(K, m.ctypes.data))
    return m[:K]


def pat_project_workspace(F: int, Cc: int) -> int:
    return int(load().pat_project_workspace(F, Cc))


def pat_project(w: torch.Tensor, masks, n_keep: int, pattern_id: Optional[torch.Tensor] = None,
                w_masked: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None):
    """w: cuda fp32 [F,C,3,3].  Returns (pattern_id u8 [F,C], w_masked fp32 [F,C,3,3])."""
    F, Cc = int(w.shape[0]), int(w.shape[1])
    m = _masks(masks)
    if pattern_id is None:
        pattern_id = torch.empty((F, Cc), dtype=torch.uint8, device=w.device)
    if w_masked is None:
        w_masked = torch.empty_like(w)
    if workspace is None:
        workspace = torch.empty(max(pat_project_workspace(F, Cc), 256), dtype=torch.uint8, device=w.device)
    _check(load().pat_project(_ptr(w), F, Cc, m.ctypes.data, len(m), int(n_keep), _ptr(pattern_id), _ptr(w_masked),
                              _ptr(workspace), workspace.numel(), _stream(stream)))
    return pattern_id, w_masked


def pat_pack_size(F: int, Cc: int, K: int, n_keep: int, dtype) -> int:
    return int(load().pat_pack_size(F, Cc, K, int(n_keep), _DT[dtype]))


def pat_blob_layout(F: int, Cc: int, K: int, n_keep: int, dtype) -> dict:
    off = (C.c_size_t * 5)()
    _check(load().pat_blob_layout(F, Cc, K, int(n_keep), _DT[dtype], off))
    return dict(zip(["perm", "fptr", "pptr", "chan", "w4"], [int(v) for v in off]))


def pat_pack(w_masked: torch.Tensor, pattern_id: torch.Tensor, masks, n_keep: int, dtype,
             blob: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    F, Cc = int(w_masked.shape[0]), int(w_masked.shape[1])
    m = _masks(masks)
    if blob is None:
        size = pat_pack_size(F, Cc, len(m), n_keep, dtype)
        if size == 0:
            raise PatError(1, "invalid pack parameters")
        blob = torch.empty(size, dtype=torch.uint8, device=w_masked.device)
    _check(load().pat_pack(_ptr(w_masked), _ptr(pattern_id), F, Cc, m.ctypes.data, len(m), int(n_keep), _DT[dtype],
                           _ptr(blob), blob.numel(), _stream(stream)))
    return blob


def pat_unpack(blob: torch.Tensor, F: int, Cc: int, masks, n_keep: int, dtype,
               out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    m = _masks(masks)
    if out is None:
        out = torch.empty((F, Cc, 3, 3), dtype=torch.float32, device=blob.device)
    _check(load().pat_unpack(_ptr(blob), F, Cc, m.ctypes.data, len(m), int(n_keep), _DT[dtype], _ptr(out), _stream(stream)))
    return out


def pat_conv3x3_workspace(F: int, Cc: int, dtype, N: int, H: int, W: int, stride: int = 1) -> int:
    """Bytes of workspace pat_conv3x3_ws wants for this layer (0: the layer runs without one)."""
    return int(load().pat_conv3x3_workspace(F, Cc, _DT[dtype], N, H, W, int(stride)))


def pat_conv3x3(blob: torch.Tensor, F: int, Cc: int, masks, n_keep: int, dtype, x: torch.Tensor,
                stride: int = 1, y: Optional[torch.Tensor] = None, stream=None,
                workspace: Optional[torch.Tensor] = None, use_workspace: bool = True, relu: bool = False,
                pool: bool = False) -> torch.Tensor:
    """x: cuda NHWC [N,H,W,C] in the blob's dtype.  Returns y NHWC [N,Ho,Wo,F]; relu / pool: pat_conv3x3_ws_act with
    act = 1 (rectifier) or act = 2 (rectifier and 2 x 2 max pooling: y is [N,H/2,W/2,F]).

    Calls pat_conv3x3_ws with `workspace` (a cuda uint8 tensor, allocated here when None and the layer wants
    one); use_workspace=False calls the entry point without workspace, pat_conv3x3."""
    m = _masks(masks)
    N, H, W = int(x.shape[0]), int(x.shape[1]), int(x.shape[2])
    if y is None:
        Ho, Wo = ((H // 2, W // 2) if pool else ((H - 1) // stride + 1, (W - 1) // stride + 1))
        y = torch.empty((N, Ho, Wo, F), dtype=x.dtype, device=x.device)
    need = pat_conv3x3_workspace(F, Cc, dtype, N, H, W, stride) if use_workspace else 0
    if relu or pool:
        # the rectifier fused into the epilogue (pat_conv3x3_ws_act; layers without workspace kernels: convolution + rectifier)
        if workspace is None:
            workspace = torch.empty(max(pat_conv3x3_workspace(F, Cc, dtype, N, H, W, stride), 256), dtype=torch.uint8, device=x.device)
        _check(load().pat_conv3x3_ws_act(_ptr(blob), F, Cc, m.ctypes.data, len(m), int(n_keep), _DT[dtype], _ptr(x), _ptr(y),
                                         N, H, W, int(stride), 2 if pool else 1, _ptr(workspace), int(workspace.numel()), _stream(stream)))
        return y
    if need == 0:
        _check(load().pat_conv3x3(_ptr(blob), F, Cc, m.ctypes.data, len(m), int(n_keep), _DT[dtype], _ptr(x), _ptr(y),
                                  N, H, W, int(stride), _stream(stream)))
        return y
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
    _check(load().pat_conv3x3_ws(_ptr(blob), F, Cc, m.ctypes.data, len(m), int(n_keep), _DT[dtype], _ptr(x), _ptr(y),
                                 N, H, W, int(stride), _ptr(workspace), int(workspace.numel()), _stream(stream)))
    return y


def pat_conv3x3_dense(w: torch.Tensor, dtype, x: torch.Tensor, stride: int = 1,
                      y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    F, Cc = int(w.shape[0]), int(w.shape[1])
    N, H, W = int(x.shape[0]), int(x.shape[1]), int(x.shape[2])
    if y is None:
        y = torch.empty((N, (H - 1) // stride + 1, (W - 1) // stride + 1, F), dtype=x.dtype, device=x.device)
    _check(load().pat_conv3x3_dense(_ptr(w), F, Cc, _DT[dtype], _ptr(x), _ptr(y), N, H, W, int(stride), _stream(stream)))
    return y


def pat_query_status(stream=None) -> int:
    rc = load().pat_query_status(_stream(stream))
    _check(rc)
    return rc


def pat_launch_count() -> int:
    return int(load().pat_launch_count())


def pat_measure_fma_peak(kind: int = 1, stream=None) -> float:
    """TFLOP/s of fma.rn.f32 (kind 0) or fma.rn.f32.f16 (kind 1) on the current device."""
    scratch = torch.empty(2 << 20, dtype=torch.uint8, device="cuda")
    out = C.c_double(0.0)
    _check(load().pat_measure_fma_peak(int(kind), _ptr(scratch), scratch.numel(), C.byref(out), _stream(stream)))
    return float(out.value)


def pat_simplex_project(d: torch.Tensor, u: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """d: cuda fp32 [n,K].  Returns u [n,K]: every row projected onto the probability simplex."""
    n, K = int(d.shape[0]), int(d.shape[1])
    if u is None:
        u = torch.empty_like(d)
    _check(load().pat_simplex_project(_ptr(d), n, K, _ptr(u), _stream(stream)))
    return u


def pat_argmax_binarize(z: torch.Tensor, index: Optional[torch.Tensor] = None, onehot: Optional[torch.Tensor] = None,
                        want_onehot: bool = True, stream=None):
    """z: cuda fp32 [n,K].  Returns (index u8 [n], onehot fp32 [n,K] or None)."""
    n, K = int(z.shape[0]), int(z.shape[1])
    if index is None:
        index = torch.empty(n, dtype=torch.uint8, device=z.device)
    if onehot is None and want_onehot:
        onehot = torch.empty_like(z)
    _check(load().pat_argmax_binarize(_ptr(z), n, K, _ptr(index), _ptr(onehot), _stream(stream)))
    return index, onehot


def pat_extract_library(w: torch.Tensor, masks, K_out: int, masks_out: Optional[torch.Tensor] = None,
                        counts: Optional[torch.Tensor] = None, stream=None):
    """w: cuda fp32 [n,3,3] (any leading shape).  Returns (masks_out int16-typed u16 bits [K_out], counts int64 [K_in]),
    both on the device."""
    m = _masks(masks)
    n = int(w.numel() // 9)
    if masks_out is None:
        masks_out = torch.empty(int(K_out), dtype=torch.int16, device=w.device)
    if counts is None:
        counts = torch.empty(len(m), dtype=torch.int64, device=w.device)
    _check(load().pat_extract_library(_ptr(w), n, m.ctypes.data, len(m), int(K_out), _ptr(masks_out), _ptr(counts),
                                      _stream(stream)))
    return masks_out, counts


def pat_relu_maxpool(x: torch.Tensor, dtype, pool: bool, y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """x: cuda NHWC.  Returns max(x, 0), 2x2 max-pooled with stride 2 when pool is set."""
    N, H, W, Cc = (int(v) for v in x.shape)
    if y is None:
        y = torch.empty((N, H // 2, W // 2, Cc) if pool else (N, H, W, Cc), dtype=x.dtype, device=x.device)
    _check(load().pat_relu_maxpool(_ptr(x), _DT[dtype], N, H, W, Cc, 1 if pool else 0, _ptr(y), _stream(stream)))
    return y


def pat_debug_set(what: int, value: int) -> None:
    _check(load().pat_debug_set(int(what), int(value)))


def pat_project_static_max_kernels() -> int:
    return int(load().pat_project_static_max_kernels())


def pat_project_static(w: torch.Tensor, masks, n_keep: int, pattern_id: torch.Tensor, w_masked: torch.Tensor, stream=None):
    """pat_project with the library's built-in scratch array: the library allocates nothing and the caller passes
    no workspace (for callers that may not allocate device memory).  Outputs must be preallocated by the caller."""
    F, Cc = int(w.shape[0]), int(w.shape[1])
    m = _masks(masks)
    _check(load().pat_project_static(_ptr(w), F, Cc, m.ctypes.data, len(m), int(n_keep), _ptr(pattern_id), _ptr(w_masked),
                                     _stream(stream)))
    return pattern_id, w_masked

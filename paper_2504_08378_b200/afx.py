"""ctypes binding of libafx: one Python function per C entry point, same names.

Argument marshalling only.  Device buffers are torch CUDA tensors (their
``data_ptr()`` is passed) or plain integer addresses; nothing is computed here and
there is no CPU path: if the CUDA library cannot be built or loaded, importing a
function from here raises.
"""
from __future__ import annotations

import ctypes
from ctypes import c_float, c_int, c_int32, c_int64, c_size_t, c_void_p

from . import build as _build

F16, BF16 = 0, 1
MODE_TOPK, MODE_THRESHOLD = 0, 1
MAX_T = 8
DTYPES = {"f16": F16, "bf16": BF16}

STATUS_NAMES = {
    0: "AFX_OK", 1: "AFX_ERR_INVALID_ARG", 2: "AFX_ERR_ALIGNMENT", 3: "AFX_ERR_CAPACITY",
    4: "AFX_ERR_UNSUPPORTED", 5: "AFX_ERR_CUDA", 6: "AFX_ERR_TIMEOUT",
}


class AfxError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {STATUS_NAMES.get(status, status)}")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads (building first if the in-tree library is missing or stale) libafx.so."""
    global _lib
    if _lib is None:
        path = _build.build_lib()
        L = ctypes.CDLL(path)
        L.afx_version.argtypes = [ctypes.POINTER(c_int), ctypes.POINTER(c_int)]
        L.afx_status_string.restype = ctypes.c_char_p
        L.afx_status_string.argtypes = [c_int32]
        L.afx_workspace_bytes.restype = c_size_t
        L.afx_workspace_bytes.argtypes = [c_int, c_int]
        L.afx_workspace_init.argtypes = [c_void_p, c_size_t, c_void_p]
        L.afx_select_active.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_float,
                                        c_void_p, c_void_p, c_void_p, c_void_p]
        L.afx_diff_active.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p,
                                      c_void_p, c_void_p]
        L.afx_sparse_gemv.argtypes = [c_void_p, c_int, c_int, c_int, c_int64, c_void_p, c_int,
                                      c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p,
                                      c_void_p]
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(fn: str, status: int):
    if status != 0:
        raise AfxError(fn, status)


def _dt(dtype):
    return DTYPES[dtype] if isinstance(dtype, str) else int(dtype)


def afx_version():
    a, b = c_int(0), c_int(0)
    _check("afx_version", lib().afx_version(ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


def afx_status_string(status: int) -> str:
    return lib().afx_status_string(int(status)).decode()


def afx_workspace_bytes(N_max: int, T_max: int = 1) -> int:
    return int(lib().afx_workspace_bytes(int(N_max), int(T_max)))


def afx_workspace_init(workspace, nbytes: int, stream=None):
    _check("afx_workspace_init", lib().afx_workspace_init(_ptr(workspace), int(nbytes), _stream(stream)))


def afx_select_active(x, dtype, K: int, T: int, mode: int, k: int, tau: float, idx, count,
                      bitmap=None, stream=None):
    _check("afx_select_active",
           lib().afx_select_active(_ptr(x), _dt(dtype), int(K), int(T), int(mode), int(k), float(tau),
                                   _ptr(idx), _ptr(count), _ptr(bitmap), _stream(stream)))


def afx_diff_active(idxA, cntA, bitmapP, K: int, miss, miss_count, hit_count, stream=None):
    _check("afx_diff_active",
           lib().afx_diff_active(_ptr(idxA), _ptr(cntA), _ptr(bitmapP), int(K), _ptr(miss),
                                 _ptr(miss_count), _ptr(hit_count), _stream(stream)))


def afx_sparse_gemv(Wt, dtype, K: int, N: int, ldw: int, x, T: int, idx, count, slot, y,
                    accumulate: int, workspace, stream=None):
    _check("afx_sparse_gemv",
           lib().afx_sparse_gemv(_ptr(Wt), _dt(dtype), int(K), int(N), int(ldw), _ptr(x), int(T),
                                 _ptr(idx), _ptr(count), _ptr(slot), _ptr(y), int(accumulate),
                                 _ptr(workspace), _stream(stream)))


def new_workspace(N_max: int, T_max: int = 1, device="cuda", stream=None):
    """Allocates (torch) and clears a GEMV workspace; returns the uint8 tensor."""
    import torch
    n = afx_workspace_bytes(N_max, T_max)
    if n == 0:
        raise AfxError("afx_workspace_bytes", 1)
    ws = torch.empty(n + 256, dtype=torch.uint8, device=device)
    off = (-ws.data_ptr()) % 256
    ws = ws[off:off + n]
    afx_workspace_init(ws, n, stream)
    return ws

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
OP_QKV, OP_O, OP_GU, OP_DOWN = 0, 1, 2, 3
XL_OFF, XL_BOOKKEEP, XL_REUSE = 0, 1, 2
BUF_H, BUF_QKV, BUF_ATTN, BUF_HM, BUF_XNORM, BUF_IDX, BUF_MISS, BUF_STATS, BUF_HINTS = range(9)
STEP_QKV, STEP_ATTN, STEP_O, STEP_GU, STEP_DOWN = range(5)
MODE_TOPK, MODE_THRESHOLD = 0, 1
MAX_T = 8
DTYPES = {"f16": F16, "bf16": BF16}

STATUS_NAMES = {
    0: "AFX_OK", 1: "AFX_ERR_INVALID_ARG", 2: "AFX_ERR_ALIGNMENT", 3: "AFX_ERR_CAPACITY",
    4: "AFX_ERR_UNSUPPORTED", 5: "AFX_ERR_CUDA", 6: "AFX_ERR_TIMEOUT",
}


class ModelDesc(ctypes.Structure):
    """afx_model_desc"""
    _fields_ = [("dtype", c_int32), ("n_layers", c_int32), ("hidden", c_int32), ("n_heads", c_int32),
                ("n_kv_heads", c_int32), ("head_dim", c_int32), ("mlp", c_int32), ("max_seq", c_int32),
                ("rms_eps", c_float), ("rope_theta", c_float), ("select_mode", c_int32),
                ("xl_depth", c_int32), ("xl_mode", c_int32)]


class LayerDesc(ctypes.Structure):
    """afx_layer_desc"""
    _fields_ = [("w_qkv", c_void_p), ("w_o", c_void_p), ("w_gu", c_void_p), ("w_down", c_void_p),
                ("g_attn", c_void_p), ("g_mlp", c_void_p), ("k_cache", c_void_p), ("v_cache", c_void_p),
                ("k", c_int32 * 4), ("tau", c_float * 4)]


class CacheDesc(ctypes.Structure):
    """afx_cache_desc"""
    _fields_ = [("dtype", c_int32), ("K", c_int32), ("N", c_int32), ("ldw", c_int64), ("capacity", c_int32),
                ("staging_rows", c_int32), ("host_base", c_void_p), ("slots", c_void_p)]


class CacheStats(ctypes.Structure):
    """afx_cache_stats"""
    _fields_ = [("hits", c_int32), ("misses", c_int32), ("transients", c_int32), ("overflow", c_int32),
                ("bytes_fetched", ctypes.c_uint64)]


class SwapDesc(ctypes.Structure):
    """afx_swap_desc"""
    _fields_ = [("dtype", c_int32), ("n_layers", c_int32), ("group", c_int32), ("K", c_int32), ("N", c_int32),
                ("ldw", c_int64), ("rows_pred", c_int32), ("rows_miss", c_int32), ("host_base", c_void_p),
                ("dev_rows", c_void_p), ("loader_stream", c_void_p)]


class SwapStats(ctypes.Structure):
    """afx_swap_stats"""
    _fields_ = [("hits", c_int32), ("ondemand", c_int32), ("overflow", c_int32), ("preloaded", c_int32),
                ("bytes_preload", ctypes.c_uint64), ("bytes_ondemand", ctypes.c_uint64)]


class CostParams(ctypes.Structure):
    """afx_cost_params"""
    _fields_ = [("sp", ctypes.c_double), ("hr", ctypes.c_double), ("si", ctypes.c_double), ("N", c_int32),
                ("n_layers", c_int32), ("S_l", ctypes.c_double), ("bw_mem", ctypes.c_double),
                ("bw_flash_small", ctypes.c_double), ("bw_flash_large", ctypes.c_double), ("M_cache", ctypes.c_double),
                ("M_kv", ctypes.c_double)]


class Cost(ctypes.Structure):
    """afx_cost"""
    _fields_ = [(n, ctypes.c_double) for n in ("M_cl", "M", "T_load", "T_comp", "T_onload", "T_preload", "T_overlap",
                                               "T_decode", "T_token")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class CostSearchIn(ctypes.Structure):
    """afx_cost_search_in"""
    _fields_ = [("S_m", ctypes.c_double), ("S_l", ctypes.c_double), ("n_layers", c_int32), ("M_max", ctypes.c_double),
                ("M_kv", ctypes.c_double), ("bw_mem", ctypes.c_double), ("bw_flash_small", ctypes.c_double),
                ("n_chunk", c_int32), ("chunk_bytes", ctypes.POINTER(ctypes.c_double)),
                ("chunk_bw", ctypes.POINTER(ctypes.c_double)), ("column_bytes", ctypes.c_double), ("n_hr", c_int32),
                ("hr_cache_frac", ctypes.POINTER(ctypes.c_double)), ("hr_value", ctypes.POINTER(ctypes.c_double)),
                ("si", ctypes.c_double), ("min_gain", ctypes.c_double), ("N_max", c_int32)]


class CostChoice(ctypes.Structure):
    """afx_cost_choice"""
    _fields_ = [("sp", ctypes.c_double), ("N", c_int32), ("M_cache", ctypes.c_double), ("hr", ctypes.c_double),
                ("bw_flash_large", ctypes.c_double), ("cost", Cost), ("stop_reason", c_int32)]


class MoeDesc(ctypes.Structure):
    """afx_moe_desc"""
    _fields_ = [("dtype", c_int32), ("hidden", c_int32), ("mlp", c_int32), ("n_experts", c_int32), ("top", c_int32),
                ("select_mode", c_int32), ("k_gu", c_int32), ("k_down", c_int32), ("tau_gu", c_float),
                ("tau_down", c_float), ("w_router", c_void_p), ("ld_router", c_int64), ("w_gu_table", c_void_p),
                ("w_down_table", c_void_p)]


class HostedOps(ctypes.Structure):
    """afx_hosted_ops"""
    _fields_ = [("cache", c_void_p * 4), ("swap", c_void_p * 4), ("slot", c_void_p * 4)]


class Q4Layer(ctypes.Structure):
    """afx_q4_layer"""
    _fields_ = [("wq", c_void_p * 4), ("ldq_bytes", c_int64 * 4)]


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
        L.afx_select_active.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_float,
                                        c_void_p, c_void_p, c_void_p, c_void_p]
        L.afx_workspace_bytes.restype = c_size_t
        L.afx_workspace_bytes.argtypes = [c_int, c_int, c_int]
        L.afx_diff_active.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p,
                                      c_void_p, c_void_p, c_void_p]
        L.afx_sparse_gemv.argtypes = [c_void_p, c_int, c_int, c_int, c_int64, c_void_p, c_int,
                                      c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p]
        L.afx_select_gemv.argtypes = [c_void_p, c_int, c_int, c_int, c_int64, c_void_p, c_int, c_int, c_int,
                                      c_float, c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
        L.afx_model_create.argtypes = [ctypes.POINTER(ModelDesc), ctypes.POINTER(LayerDesc),
                                       ctypes.POINTER(c_void_p)]
        L.afx_model_destroy.argtypes = [c_void_p]
        L.afx_state_bytes.restype = c_size_t
        L.afx_state_bytes.argtypes = [c_void_p, c_int]
        L.afx_state_create.argtypes = [c_void_p, c_int, c_void_p, c_size_t, c_void_p,
                                       ctypes.POINTER(c_void_p)]
        L.afx_state_destroy.argtypes = [c_void_p]
        L.afx_state_buffer.argtypes = [c_void_p, c_int, c_int, ctypes.POINTER(c_void_p),
                                       ctypes.POINTER(c_size_t)]
        L.afx_layer_step.argtypes = [c_void_p, c_int, c_void_p, c_int, c_void_p]
        L.afx_layer_kernel.argtypes = [c_void_p, c_int, c_void_p, c_int, c_int, c_void_p]
        L.afx_mlp_block.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
        L.afx_cache_create.argtypes = [ctypes.POINTER(CacheDesc), ctypes.POINTER(c_void_p)]
        L.afx_cache_destroy.argtypes = [c_void_p]
        L.afx_cache_reset.argtypes = [c_void_p, c_void_p]
        L.afx_cache_install.argtypes = [c_void_p, c_void_p, c_int, c_void_p]
        L.afx_cache_fetch.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.afx_cache_snapshot.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p]
        L.afx_swap_host_offset.restype = c_size_t
        L.afx_swap_host_offset.argtypes = [c_int, c_int, c_int, c_int64, c_int, c_int]
        L.afx_swap_pack_host.argtypes = [ctypes.POINTER(c_void_p), c_int, c_int, c_int, c_int64, c_void_p]
        L.afx_swap_device_bytes.restype = c_size_t
        L.afx_swap_device_bytes.argtypes = [ctypes.POINTER(SwapDesc)]
        L.afx_swap_create.argtypes = [ctypes.POINTER(SwapDesc), ctypes.POINTER(c_void_p)]
        L.afx_swap_destroy.argtypes = [c_void_p]
        L.afx_swap_preload.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_int, c_void_p, c_void_p]
        L.afx_swap_acquire.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                       ctypes.POINTER(c_void_p)]
        L.afx_cost_eval.argtypes = [ctypes.POINTER(CostParams), ctypes.POINTER(Cost)]
        L.afx_cost_search.argtypes = [ctypes.POINTER(CostSearchIn), ctypes.POINTER(CostChoice)]
        L.afx_moe_workspace_bytes.restype = c_size_t
        L.afx_moe_workspace_bytes.argtypes = [ctypes.POINTER(MoeDesc)]
        L.afx_moe_block.argtypes = [ctypes.POINTER(MoeDesc), c_void_p, c_void_p, c_int, c_void_p, c_size_t, c_void_p]
        L.afx_q4_row_bytes.restype = c_size_t
        L.afx_q4_row_bytes.argtypes = [c_int]
        L.afx_sparse_gemv_q4.argtypes = [c_void_p, c_int, c_int, c_int64, c_void_p, c_int, c_void_p, c_void_p, c_void_p,
                                         c_int, c_void_p, c_void_p]
        L.afx_layer_step_hosted.argtypes = [c_void_p, c_int, c_void_p, c_int, ctypes.POINTER(HostedOps), c_void_p, c_void_p]
        L.afx_layer_step_q4.argtypes = [c_void_p, c_int, c_void_p, c_int, ctypes.POINTER(Q4Layer), c_void_p, c_void_p]
        L.afx_mlp_block_noalloc.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_int, c_int, c_int,
                                            c_float, c_int, c_float, c_void_p, c_void_p]
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


def afx_select_active(x, dtype, K: int, T: int, mode: int, k: int, tau: float, idx, count,
                      bitmap=None, stream=None):
    _check("afx_select_active",
           lib().afx_select_active(_ptr(x), _dt(dtype), int(K), int(T), int(mode), int(k), float(tau),
                                   _ptr(idx), _ptr(count), _ptr(bitmap), _stream(stream)))


def afx_workspace_bytes(K_max: int, N_max: int, T_max: int) -> int:
    return int(lib().afx_workspace_bytes(int(K_max), int(N_max), int(T_max)))


def afx_diff_active(idxA, cntA, bitmapP, K: int, miss, miss_count, hit_count, stream=None, dev_status=None):
    _check("afx_diff_active",
           lib().afx_diff_active(_ptr(idxA), _ptr(cntA), _ptr(bitmapP), int(K), _ptr(miss),
                                 _ptr(miss_count), _ptr(hit_count), _ptr(dev_status), _stream(stream)))


def afx_sparse_gemv(Wt, dtype, K: int, N: int, ldw: int, x, T: int, idx, count, slot, y,
                    accumulate: int, stream=None, dev_status=None):
    _check("afx_sparse_gemv",
           lib().afx_sparse_gemv(_ptr(Wt), _dt(dtype), int(K), int(N), int(ldw), _ptr(x), int(T),
                                 _ptr(idx), _ptr(count), _ptr(slot), _ptr(y), int(accumulate),
                                 _ptr(dev_status), _stream(stream)))


def afx_select_gemv(Wt, dtype, K: int, N: int, ldw: int, x, T: int, mode: int, k: int, tau: float, y,
                    accumulate: int, idx_out=None, count_out=None, stream=None, kth_hint=None):
    _check("afx_select_gemv",
           lib().afx_select_gemv(_ptr(Wt), _dt(dtype), int(K), int(N), int(ldw), _ptr(x), int(T), int(mode),
                                 int(k), float(tau), _ptr(y), int(accumulate), _ptr(idx_out), _ptr(count_out),
                                 _ptr(kth_hint), _stream(stream)))


def afx_model_create(desc: ModelDesc, layers) -> int:
    """layers: sequence of LayerDesc (len == desc.n_layers).  Returns the model handle."""
    arr = (LayerDesc * len(layers))(*layers)
    out = c_void_p(0)
    _check("afx_model_create", lib().afx_model_create(ctypes.byref(desc), arr, ctypes.byref(out)))
    return out.value


def afx_model_destroy(model: int):
    _check("afx_model_destroy", lib().afx_model_destroy(model))


def afx_state_bytes(model: int, T: int) -> int:
    return int(lib().afx_state_bytes(model, int(T)))


def afx_state_create(model: int, T: int, blob, nbytes: int, stream=None) -> int:
    out = c_void_p(0)
    _check("afx_state_create",
           lib().afx_state_create(model, int(T), _ptr(blob), int(nbytes), _stream(stream), ctypes.byref(out)))
    return out.value


def afx_state_destroy(state: int):
    _check("afx_state_destroy", lib().afx_state_destroy(state))


def afx_state_buffer(state: int, which: int, op: int = 0):
    """Returns (device address, bytes) of a buffer inside the state blob."""
    ptr, n = c_void_p(0), c_size_t(0)
    _check("afx_state_buffer", lib().afx_state_buffer(state, int(which), int(op), ctypes.byref(ptr), ctypes.byref(n)))
    return ptr.value, n.value


def afx_layer_step(model: int, layer: int, state: int, pos: int, stream=None):
    _check("afx_layer_step", lib().afx_layer_step(model, int(layer), state, int(pos), _stream(stream)))


def afx_layer_kernel(model: int, layer: int, state: int, pos: int, which: int, stream=None):
    _check("afx_layer_kernel", lib().afx_layer_kernel(model, int(layer), state, int(pos), int(which), _stream(stream)))


def afx_mlp_block(model: int, layer: int, state: int, x, y, stream=None):
    _check("afx_mlp_block", lib().afx_mlp_block(model, int(layer), state, _ptr(x), _ptr(y), _stream(stream)))


def afx_mlp_block_noalloc(w_gu, w_down, dtype, hidden: int, mlp: int, x, T: int, mode: int, k_gu: int, tau_gu: float,
                          k_down: int, tau_down: float, y, stream=None):
    """The MLP block for callers that may not allocate device memory: no model object, no state
    blob; the intermediate vector lives in a fixed 512 KB array inside the library (shared by all
    calls on a device, so calls that overlap on the GPU race).  mlp <= 32768."""
    _check("afx_mlp_block_noalloc",
           lib().afx_mlp_block_noalloc(_ptr(w_gu), _ptr(w_down), _dt(dtype), int(hidden), int(mlp), _ptr(x), int(T),
                                       int(mode), int(k_gu), float(tau_gu), int(k_down), float(tau_down), _ptr(y),
                                       _stream(stream)))


def afx_cache_create(desc: CacheDesc) -> int:
    out = c_void_p(0)
    _check("afx_cache_create", lib().afx_cache_create(ctypes.byref(desc), ctypes.byref(out)))
    return out.value


def afx_cache_destroy(cache: int):
    _check("afx_cache_destroy", lib().afx_cache_destroy(cache))


def afx_cache_reset(cache: int, stream=None):
    _check("afx_cache_reset", lib().afx_cache_reset(cache, _stream(stream)))


def afx_cache_install(cache: int, channels, stream=None):
    """channels: sequence of channel ids (host side) pre-loaded into the lowest free slots."""
    arr = (c_int32 * len(channels))(*[int(c) for c in channels])
    _check("afx_cache_install", lib().afx_cache_install(cache, arr, len(channels), _stream(stream)))


def afx_cache_fetch(cache: int, idx, count, slot_out, stats=None, stream=None, dev_status=None):
    _check("afx_cache_fetch",
           lib().afx_cache_fetch(cache, _ptr(idx), _ptr(count), _ptr(slot_out), _ptr(stats), _ptr(dev_status),
                                 _stream(stream)))


def afx_cache_snapshot(cache: int, K: int, stream=None):
    """Returns (slot_of[K] int32, usage[K] uint32) as numpy arrays."""
    import numpy as np
    slot_of = np.empty(K, np.int32)
    usage = np.empty(K, np.uint32)
    _check("afx_cache_snapshot",
           lib().afx_cache_snapshot(cache, slot_of.ctypes.data, usage.ctypes.data, _stream(stream)))
    return slot_of, usage


def afx_swap_host_offset(n_layers: int, group: int, K: int, ldw: int, layer: int, channel: int) -> int:
    """Element offset of (layer, channel) in the cross-layer-group host image (host arithmetic)."""
    v = int(lib().afx_swap_host_offset(int(n_layers), int(group), int(K), int(ldw), int(layer), int(channel)))
    if v == (1 << 64) - 1:
        raise AfxError("afx_swap_host_offset", 1)
    return v


def afx_swap_pack_host(per_layer_ptrs, n_layers: int, group: int, K: int, ldw: int, host_out):
    """per_layer_ptrs: host addresses of the per-layer [K][ldw] tensors; host_out: host address."""
    arr = (c_void_p * n_layers)(*[int(p) for p in per_layer_ptrs])
    _check("afx_swap_pack_host", lib().afx_swap_pack_host(arr, int(n_layers), int(group), int(K), int(ldw), host_out))


def afx_swap_device_bytes(desc: SwapDesc) -> int:
    return int(lib().afx_swap_device_bytes(ctypes.byref(desc)))


def afx_swap_create(desc: SwapDesc) -> int:
    out = c_void_p(0)
    _check("afx_swap_create", lib().afx_swap_create(ctypes.byref(desc), ctypes.byref(out)))
    return out.value


def afx_swap_destroy(swap: int):
    _check("afx_swap_destroy", lib().afx_swap_destroy(swap))


def afx_swap_preload(swap: int, group_index: int, idxP, cntP, copy_blocks: int = 0, stream=None, dev_status=None):
    _check("afx_swap_preload", lib().afx_swap_preload(swap, int(group_index), _ptr(idxP), _ptr(cntP), int(copy_blocks),
                                                      _ptr(dev_status), _stream(stream)))


def afx_swap_acquire(swap: int, layer: int, idxA, cntA, slot_out, stats=None, stream=None, dev_status=None) -> int:
    """Returns the device address of the layer's rows (the Wt argument of afx_sparse_gemv)."""
    rows = c_void_p(0)
    _check("afx_swap_acquire", lib().afx_swap_acquire(swap, int(layer), _ptr(idxA), _ptr(cntA), _ptr(slot_out),
                                                      _ptr(stats), _ptr(dev_status), _stream(stream), ctypes.byref(rows)))
    return rows.value


def afx_cost_eval(**kw) -> dict:
    """Eq. 1-9 for the given afx_cost_params fields; returns the afx_cost fields as a dict."""
    out = Cost()
    _check("afx_cost_eval", lib().afx_cost_eval(ctypes.byref(CostParams(**kw)), ctypes.byref(out)))
    return out.as_dict()


def afx_cost_search(chunk_table, hr_table, **kw) -> dict:
    """chunk_table: [(chunk bytes, bytes/s)], hr_table: [(cache size / S_m, hit rate)], both
    ascending; the other afx_cost_search_in fields by keyword."""
    cb = (ctypes.c_double * len(chunk_table))(*[float(a) for a, _ in chunk_table])
    cw = (ctypes.c_double * len(chunk_table))(*[float(b) for _, b in chunk_table])
    hf = (ctypes.c_double * len(hr_table))(*[float(a) for a, _ in hr_table])
    hv = (ctypes.c_double * len(hr_table))(*[float(b) for _, b in hr_table])
    arg = CostSearchIn(n_chunk=len(chunk_table), chunk_bytes=cb, chunk_bw=cw, n_hr=len(hr_table), hr_cache_frac=hf,
                       hr_value=hv, **kw)
    out = CostChoice()
    _check("afx_cost_search", lib().afx_cost_search(ctypes.byref(arg), ctypes.byref(out)))
    return dict(sp=out.sp, N=out.N, M_cache=out.M_cache, hr=out.hr, bw_flash_large=out.bw_flash_large,
                stop_reason=out.stop_reason, cost=out.cost.as_dict())


def afx_moe_workspace_bytes(desc: MoeDesc) -> int:
    return int(lib().afx_moe_workspace_bytes(ctypes.byref(desc)))


def afx_moe_block(desc: MoeDesc, x, y, accumulate: int, workspace, workspace_bytes: int, stream=None):
    _check("afx_moe_block", lib().afx_moe_block(ctypes.byref(desc), _ptr(x), _ptr(y), int(accumulate), _ptr(workspace),
                                                int(workspace_bytes), _stream(stream)))


def afx_q4_row_bytes(N: int) -> int:
    return int(lib().afx_q4_row_bytes(int(N)))


def afx_sparse_gemv_q4(Wq, K: int, N: int, ldq_bytes: int, x, x_dtype, idx, count, y, accumulate: int, stream=None,
                       dev_status=None):
    _check("afx_sparse_gemv_q4",
           lib().afx_sparse_gemv_q4(_ptr(Wq), int(K), int(N), int(ldq_bytes), _ptr(x), _dt(x_dtype), _ptr(idx), _ptr(count),
                                    _ptr(y), int(accumulate), _ptr(dev_status), _stream(stream)))


def afx_layer_step_q4(model: int, layer: int, state: int, pos: int, q4: Q4Layer, stream=None, dev_status=None):
    _check("afx_layer_step_q4", lib().afx_layer_step_q4(model, int(layer), state, int(pos), ctypes.byref(q4),
                                                        _ptr(dev_status), _stream(stream)))


def afx_layer_step_hosted(model: int, layer: int, state: int, pos: int, ops: HostedOps, stream=None, dev_status=None):
    _check("afx_layer_step_hosted", lib().afx_layer_step_hosted(model, int(layer), state, int(pos), ctypes.byref(ops),
                                                                _ptr(dev_status), _stream(stream)))

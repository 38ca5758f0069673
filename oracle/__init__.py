"""CPU oracle for the active-weight hot path (test infrastructure only).

A thin ctypes front for ``afx_oracle.c`` plus the decoder-layer composition in
``oracle.layer``.  Nothing here is part of the product: only the tests, the smoke
check and the benchmark's CPU-baseline leg may import it, and it imports nothing
from the CUDA package.  Arrays of 16-bit floats are numpy ``uint16`` bit patterns;
``dtype`` is ``"f16"`` or ``"bf16"``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "afx_oracle.c")
_SO = os.path.join(_HERE, "libafx_oracle.so")

DTYPES = {"f16": 0, "bf16": 1}
TOPK, THRESHOLD = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP only spreads independent output rows)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _SO)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def threads() -> int:
    return int(lib().afxo_threads())


def set_threads(n: int) -> None:
    """Caps the oracle's worker threads (for a one-core timing); results do not depend on it."""
    lib().afxo_set_threads(int(n))


def decode(bits, dtype: str) -> np.ndarray:
    """fp64 values of 16-bit patterns."""
    bits = _u16(bits)
    out = np.empty(bits.shape, np.float64)
    lib().afxo_decode(_p(bits, ctypes.c_uint16), ctypes.c_int64(bits.size), DTYPES[dtype],
                      _p(out, ctypes.c_double))
    return out


def round_to(values, dtype: str) -> np.ndarray:
    """Round fp64 values once (nearest-even) to 16-bit patterns."""
    v = np.ascontiguousarray(values, np.float64)
    out = np.empty(v.shape, np.uint16)
    lib().afxo_round(_p(v, ctypes.c_double), ctypes.c_int64(v.size), DTYPES[dtype],
                     _p(out, ctypes.c_uint16))
    return out


def select_active(x, dtype: str, mode: int, k: int = 0, tau: float = 0.0) -> np.ndarray:
    """Ascending active-channel list of x[T][K] (union over the T tokens)."""
    x = _u16(x)
    if x.ndim == 1:
        x = x[None, :]
    T, K = x.shape
    idx = np.empty(K, np.int32)
    cnt = ctypes.c_int32(0)
    rc = lib().afxo_select_active(_p(x, ctypes.c_uint16), DTYPES[dtype], K, T, mode, int(k),
                                  ctypes.c_float(tau), _p(idx, ctypes.c_int32),
                                  ctypes.byref(cnt))
    if rc != 0:
        raise ValueError("afxo_select_active: bad argument")
    return idx[: cnt.value].copy()


def diff_active(idxA, idxP, K: int):
    """(miss = A \\ P ascending, hit = |A & P|) for ascending lists A, P."""
    A = np.ascontiguousarray(idxA, np.int32)
    P = np.ascontiguousarray(idxP, np.int32)
    miss = np.empty(max(A.size, 1), np.int32)
    nm, nh = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = lib().afxo_diff_active(_p(A, ctypes.c_int32), A.size, _p(P, ctypes.c_int32), P.size, K,
                                _p(miss, ctypes.c_int32), ctypes.byref(nm), ctypes.byref(nh))
    if rc != 0:
        raise ValueError("afxo_diff_active: bad argument")
    return miss[: nm.value].copy(), nh.value


def sparse_gemv(Wt, dtype: str, N: int, x, idx, slot=None) -> np.ndarray:
    """y[T][N] (fp64) = sum_c x[t][idx[c]] * Wt[col(c)][:N]; Wt is [rows][ldw] bit patterns."""
    Wt = _u16(Wt)
    x = _u16(x)
    if x.ndim == 1:
        x = x[None, :]
    T, K = x.shape
    ldw = Wt.shape[1]
    idx = np.ascontiguousarray(idx, np.int32)
    y = np.empty((T, N), np.float64)
    sp = None
    if slot is not None:
        slot = np.ascontiguousarray(slot, np.int32)
        sp = _p(slot, ctypes.c_int32)
    rc = lib().afxo_sparse_gemv(_p(Wt, ctypes.c_uint16), DTYPES[dtype], K, N,
                                ctypes.c_int64(ldw), _p(x, ctypes.c_uint16), T,
                                _p(idx, ctypes.c_int32), idx.size, sp, _p(y, ctypes.c_double))
    if rc != 0:
        raise ValueError("afxo_sparse_gemv: bad argument")
    return y


def rmsnorm(h, g, eps: float, dtype: str) -> np.ndarray:
    h = np.ascontiguousarray(h, np.float64)
    if h.ndim == 1:
        h = h[None, :]
    g = np.ascontiguousarray(g, np.float64)
    T, H = h.shape
    out = np.empty((T, H), np.uint16)
    lib().afxo_rmsnorm(_p(h, ctypes.c_double), _p(g, ctypes.c_double), T, H, ctypes.c_double(eps),
                       DTYPES[dtype], _p(out, ctypes.c_uint16))
    return out


def rope(v, pos, theta: float = 10000.0) -> np.ndarray:
    """Rotate v[T][heads][D] (fp64) by the positions pos[T]; returns a new array."""
    v = np.array(v, np.float64, order="C", copy=True)
    T, heads, D = v.shape
    pos = np.ascontiguousarray(pos, np.int32)
    lib().afxo_rope(_p(v, ctypes.c_double), T, heads, D, _p(pos, ctypes.c_int32),
                    ctypes.c_double(theta))
    return v


def attention(q, kc, vc, L: int, dtype: str) -> np.ndarray:
    """q[q_heads][D] fp64, kc/vc [>=L][kv_heads][D] fp16 bits -> out[q_heads][D] dtype bits."""
    q = np.ascontiguousarray(q, np.float64)
    kc, vc = _u16(kc), _u16(vc)
    q_heads, D = q.shape
    kv_heads = kc.shape[1]
    out = np.empty((q_heads, D), np.uint16)
    lib().afxo_attention(_p(q, ctypes.c_double), _p(kc, ctypes.c_uint16), _p(vc, ctypes.c_uint16),
                         L, q_heads, kv_heads, D, DTYPES[dtype], _p(out, ctypes.c_uint16))
    return out


def silu_mul(g, u, dtype: str) -> np.ndarray:
    g = np.ascontiguousarray(g, np.float64)
    u = np.ascontiguousarray(u, np.float64)
    out = np.empty(g.shape, np.uint16)
    lib().afxo_silu_mul(_p(g, ctypes.c_double), _p(u, ctypes.c_double), ctypes.c_int64(g.size),
                        DTYPES[dtype], _p(out, ctypes.c_uint16))
    return out


class LfuCache:
    """Context-level LFU column cache of one weight tensor (Sec. 4.2), state on the host."""

    def __init__(self, K: int, capacity: int):
        self.K, self.C = int(K), int(capacity)
        self.slot_of = np.full(K, -1, np.int32)
        self.chan_of = np.full(capacity, -1, np.int32)
        self.freq = np.zeros(K, np.uint32)

    def reset_counts(self):
        """New sequence: the usage count of every channel starts from zero."""
        self.freq[:] = 0

    def install(self, channels):
        """Pre-load channels into the lowest free slots (initial cache contents)."""
        for j in channels:
            s = int(np.flatnonzero(self.chan_of < 0)[0])
            self.chan_of[s] = j
            self.slot_of[j] = s

    def step(self, idx):
        """Returns dict(slot, fetched, hits, misses, transients) for one token's active list."""
        idx = np.ascontiguousarray(idx, np.int32)
        slot = np.empty(max(idx.size, 1), np.int32)
        fetched = np.empty(max(idx.size, 1), np.int32)
        nh, nm, nt = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
        rc = lib().afxo_cache_step(self.K, self.C, _p(self.slot_of, ctypes.c_int32),
                                   _p(self.chan_of, ctypes.c_int32),
                                   _p(self.freq, ctypes.c_uint32), _p(idx, ctypes.c_int32),
                                   idx.size, _p(slot, ctypes.c_int32),
                                   _p(fetched, ctypes.c_int32), ctypes.byref(nh),
                                   ctypes.byref(nm), ctypes.byref(nt))
        if rc != 0:
            raise ValueError("afxo_cache_step: bad argument")
        return dict(slot=slot[: idx.size].copy(), fetched=fetched[: nm.value].copy(),
                    hits=nh.value, misses=nm.value, transients=nt.value)

    def cached(self) -> np.ndarray:
        return np.sort(self.chan_of[self.chan_of >= 0])


# ---- cross-layer-group preloading (Sec. 3 "Data layout", Sec. 4 operations PL and L) ----

def group_layout_offset(layer: int, channel: int, n_layers: int, d: int, K: int, ldw: int) -> int:
    """Element offset of (layer, channel) of ONE operator type in the reordered host image
    (Sec. 3 "Data layout", Fig. "reordered weights in a 4-layers group"): groups in layer order;
    inside a group the order is channel id, then layer id:
    [Ch0_L, Ch0_L+1, .., Ch0_L+d-1, Ch1_L, ..].  A group of dg layers (dg = d except for a
    shorter last group) therefore stores channel j as one run of dg columns."""
    g, i = layer // d, layer % d
    dg = min(d, n_layers - g * d)
    return ((g * d * K) + channel * dg + i) * ldw   # all earlier groups are full: g*d layers * K columns


def pack_group_layout(per_layer, d: int) -> np.ndarray:
    """per_layer: list of [K][ldw] uint16 arrays (one operator type, layer order) -> the host
    image in the layout of group_layout_offset, written with plain loops over its definition."""
    L = len(per_layer)
    K, ldw = per_layer[0].shape
    out = np.empty(L * K * ldw, np.uint16)
    for l in range(L):
        for j in range(K):
            o = group_layout_offset(l, j, L, d, K, ldw)
            out[o:o + ldw] = per_layer[l][j]
    return out


def swap_acquire(P, A, rows_pred: int, rows_miss: int):
    """Where each active channel of a layer is found after the preload of its group (Sec. 3:
    what the prediction covered was preloaded, "the missed active weights during preloading will
    be on-demand loaded"): the c-th predicted channel sits in row c (c < rows_pred; predicted
    channels beyond rows_pred were not preloaded); a channel of A that was not preloaded is
    loaded on demand into row rows_pred + m, m = its rank among this layer's on-demand loads,
    or gets -1 when rows_miss is exhausted.  Returns dict(slot, ondemand, hits, overflow)."""
    P = [int(j) for j in P][:rows_pred]
    row_of = {j: c for c, j in enumerate(P)}
    slot, ondemand, overflow = [], [], 0
    for j in (int(v) for v in A):
        if j in row_of:
            slot.append(row_of[j])
        else:
            m = len(ondemand) + overflow
            if m < rows_miss:
                slot.append(rows_pred + m)
                ondemand.append(j)
            else:
                slot.append(-1)
                overflow += 1
    return dict(slot=np.array(slot, np.int32), ondemand=np.array(ondemand, np.int32),
                hits=len(slot) - len(ondemand) - overflow, overflow=overflow)


# ---- cost model of the swapping pipeline (Sec. 4.1, Eq. 1-9) ----

def cost_model(sp, hr, si, N, S_l, bw_mem, bw_flash_small, bw_flash_large, M_cache=0.0, M_kv=0.0, n_layers=None):
    """Eq. 1-9 written out one by one, in the paper's symbols (sizes in bytes, bandwidths in
    bytes/s, times in s).  T_decode is Eq. 1 as printed: the first group's load, ONE overlap
    stage and the last group's computation.  With n_layers given, T_token also counts one
    overlap stage per further group (n_layers / N groups: first load, groups - 1 overlap
    stages, last computation)."""
    M_cl = S_l * (1.0 - sp) * N                                            # Eq. 9
    M = M_cl + M_cache + M_kv                                              # Eq. 8
    T_load = M_cl * (1.0 - hr) / bw_flash_small                            # Eq. 3
    T_comp = M_cl / bw_mem                                                 # Eq. 4
    T_onload = S_l * (1.0 - sp) * (1.0 - hr) * (1.0 - si) / bw_flash_small  # Eq. 6
    T_preload = M_cl * (1.0 - hr) / bw_flash_large                         # Eq. 7
    T_overlap = T_onload + max(T_preload, T_comp)                          # Eq. 5
    T_decode = T_load + T_overlap + T_comp                                 # Eq. 1
    out = dict(M_cl=M_cl, M=M, T_load=T_load, T_comp=T_comp, T_onload=T_onload, T_preload=T_preload,
               T_overlap=T_overlap, T_decode=T_decode)
    if n_layers is not None:
        groups = -(-n_layers // N)
        out["T_token"] = T_load + (groups - 1) * T_overlap + T_comp
    return out


# ---- 4-bit block-quantised weights (Sec. 6: the channel's scales travel with the channel) ----

def q4_decode_loops(rows, N: int) -> np.ndarray:
    """fp64 values [K][N] of channel-contiguous 4-bit rows: per channel N/2 bytes of codes, then
    N/32 fp16 scales; block b = outputs 32b .. 32b+31, byte m of the block holds the code of
    output 32b + m in its low 4 bits and of output 32b + 16 + m in its high 4 bits; value =
    (code - 8) * scale.  Plain loops over that definition (small inputs)."""
    rows = np.ascontiguousarray(rows, np.uint8)
    K = rows.shape[0]
    out = np.empty((K, N), np.float64)
    for j in range(K):
        scales = decode(rows[j, N // 2: N // 2 + N // 16].copy().view(np.uint16), "f16")
        for b in range(N // 32):
            blk = rows[j, 16 * b: 16 * b + 16]
            for m in range(16):
                out[j, 32 * b + m] = (int(blk[m] & 0x0F) - 8) * scales[b]
                out[j, 32 * b + 16 + m] = (int(blk[m] >> 4) - 8) * scales[b]
    return out


def q4_decode(rows, N: int) -> np.ndarray:
    """The same decoding with whole-array numpy operations (for inputs of real size; the tests
    hold it equal to q4_decode_loops)."""
    rows = np.ascontiguousarray(rows, np.uint8)
    K = rows.shape[0]
    codes = rows[:, : N // 2].reshape(K, N // 32, 16)
    q = np.concatenate([codes & 0x0F, codes >> 4], axis=2).astype(np.float64)     # [K][block][32]
    scales = decode(rows[:, N // 2: N // 2 + N // 16].copy().view(np.uint16), "f16")  # [K][block]
    return ((q - 8.0) * scales[:, :, None]).reshape(K, N)


def sparse_gemv_q4(rows, N: int, x, dtype: str, idx) -> np.ndarray:
    """y[N] (fp64) = sum_c x[idx[c]] * W[idx[c]][:], W = q4_decode(rows), ascending c."""
    xv = decode(np.asarray(x, np.uint16).reshape(-1), dtype)
    idx = np.asarray(idx, np.int64)
    W = q4_decode(np.asarray(rows)[idx], N) if idx.size else np.zeros((0, N))
    y = np.zeros(N)
    for c in range(idx.size):
        y += xv[idx[c]] * W[c]
    return y[None, :]

"""Seeded synthetic inputs shared by the CUDA path's tests, the oracle's tests and the bench.

This module only *draws inputs*: random weights, activations, caches and channel
activity patterns with the shapes and value distributions of the Llama-shaped
decode workloads.  It holds none of the method's arithmetic (no selection, no
GEMV, no cache policy) and imports neither the CUDA binding nor the oracle.

All 16-bit float arrays are numpy ``uint16`` bit patterns; ``dtype`` is ``"f16"``
(IEEE binary16) or ``"bf16"``.  Streams are Philox counters keyed by
``(seed, stream id)``, so any tensor can be regenerated on its own.
"""
from __future__ import annotations

import numpy as np

DTYPES = ("f16", "bf16")


def rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream) & (2**64 - 1)]))


def f32_to_bits(a, dtype: str) -> np.ndarray:
    """Round float32 values to nearest-even 16-bit patterns."""
    a = np.ascontiguousarray(a, np.float32)
    if dtype == "f16":
        return a.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        u = a.view(np.uint32)
        nan = np.isnan(a)
        r = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)
        if nan.any():
            r = np.where(nan, np.uint16(0x7FC0), r)
        return r
    raise ValueError(dtype)


def bits_to_f32(bits, dtype: str) -> np.ndarray:
    bits = np.ascontiguousarray(bits, np.uint16)
    if dtype == "f16":
        return bits.view(np.float16).astype(np.float32)
    if dtype == "bf16":
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    raise ValueError(dtype)


def normal_bits(seed: int, stream: int, shape, sigma: float, dtype: str) -> np.ndarray:
    """N(0, sigma^2) values rounded to dtype; used for weights and KV caches."""
    g = rng(seed, stream)
    a = g.standard_normal(size=shape, dtype=np.float32)
    a *= np.float32(sigma)
    return f32_to_bits(a, dtype)


def weight(seed: int, stream: int, K: int, N: int, dtype: str, sigma: float = 0.02,
           ldw: int | None = None) -> np.ndarray:
    """Channel-contiguous operator weight Wt[K][ldw]; columns N..ldw are zero padding."""
    ldw = N if ldw is None else ldw
    w = normal_bits(seed, stream, (K, N), sigma, dtype)
    if ldw == N:
        return w
    out = np.zeros((K, ldw), np.uint16)
    out[:, :N] = w
    return out


def laplace(seed: int, stream: int, shape, scale: float = 1.0) -> np.ndarray:
    """Laplace(0, scale) by inverse CDF of seeded uniforms (float64)."""
    u = rng(seed, stream).random(size=shape) - 0.5
    return -scale * np.sign(u) * np.log1p(-2.0 * np.abs(u))


def laplace_bits(seed: int, stream: int, shape, dtype: str, scale: float = 1.0) -> np.ndarray:
    return f32_to_bits(laplace(seed, stream, shape, scale).astype(np.float32), dtype)


def laplace_tau(p: float, scale: float = 1.0) -> float:
    """Magnitude below which a fraction p of Laplace(0, scale) draws fall (|x| ~ Exp(1/scale)).

    p = 0 returns -1, the "keep every channel" setting of the threshold mode.
    """
    if p <= 0.0:
        return -1.0
    return float(-scale * np.log1p(-p))


def keep_count(K: int, sparsity_percent: int) -> int:
    """Channels kept at an integer sparsity percentage: K - floor(K * p / 100)."""
    return int(K - (K * int(sparsity_percent)) // 100)


def channel_scales(seed: int, stream: int, K: int, sigma: float = 0.5) -> np.ndarray:
    """Persistent per-channel lognormal scale: gives successive layers similar |x| profiles."""
    return np.exp(sigma * rng(seed, stream).standard_normal(K))


def zipf_activity_bits(seed: int, stream: int, K: int, dtype: str, alpha: float = 1.1,
                       perm_stream: int = 0) -> np.ndarray:
    """One activation vector whose top-k sets follow a Zipf(alpha) channel popularity.

    Channel weights w_r ~ r^-alpha are laid over a seeded permutation shared by all steps
    of a tensor (``perm_stream``); score_j = ln w_j + Gumbel noise, so the k largest scores
    are a weighted sample without replacement.  |x_j| = exp(score_j / 4) keeps the values
    inside fp16/bf16 range while preserving the order; signs are random.
    """
    perm = rng(seed, perm_stream).permutation(K)
    rank = np.empty(K, np.int64)
    rank[perm] = np.arange(1, K + 1)
    g = rng(seed, stream)
    score = -alpha * np.log(rank.astype(np.float64)) + g.gumbel(size=K)
    mag = np.exp(score / 4.0)
    sign = np.where(g.random(K) < 0.5, -1.0, 1.0)
    return f32_to_bits((mag * sign).astype(np.float32), dtype)


def interleave_gate_up(w_gate: np.ndarray, w_up: np.ndarray) -> np.ndarray:
    """[K][mlp] gate and up -> [K][2*mlp] with columns in groups of 16: gate[8m..8m+8) then
    up[8m..8m+8) (the storage layout of the fused gate/up operator; a pure re-arrangement)."""
    K, M = w_gate.shape
    assert w_up.shape == (K, M) and M % 8 == 0
    out = np.empty((K, M // 8, 2, 8), w_gate.dtype)
    out[:, :, 0, :] = w_gate.reshape(K, M // 8, 8)
    out[:, :, 1, :] = w_up.reshape(K, M // 8, 8)
    return out.reshape(K, 2 * M)


def layer_weights(seed: int, layer: int, hidden: int, n_heads: int, n_kv_heads: int, mlp: int,
                  dtype: str, head_dim: int = 128, sigma: float = 0.02, gain_jitter: float = 0.0) -> dict:
    """Random-init weights of one Llama-shaped decoder layer (bit patterns, channel-contiguous)."""
    base = 1000 * (layer + 1)
    n_qkv = (n_heads + 2 * n_kv_heads) * head_dim
    g = rng(seed, base + 7)
    return dict(
        w_qkv=weight(seed, base + 1, hidden, n_qkv, dtype, sigma),
        w_o=weight(seed, base + 2, n_heads * head_dim, hidden, dtype, sigma),
        w_gate=weight(seed, base + 3, hidden, mlp, dtype, sigma),
        w_up=weight(seed, base + 4, hidden, mlp, dtype, sigma),
        w_down=weight(seed, base + 5, mlp, hidden, dtype, sigma),
        g_attn=(1.0 + gain_jitter * g.standard_normal(hidden)).astype(np.float32),
        g_mlp=(1.0 + gain_jitter * g.standard_normal(hidden)).astype(np.float32),
    )


def kv_cache(seed: int, layer: int, T: int, max_seq: int, n_kv_heads: int, filled: int,
             head_dim: int = 128):
    """fp16 K and V caches [T][max_seq][n_kv_heads][head_dim] with `filled` past rows ~ N(0,1)."""
    kc = np.zeros((T, max_seq, n_kv_heads, head_dim), np.uint16)
    vc = np.zeros((T, max_seq, n_kv_heads, head_dim), np.uint16)
    kc[:, :filled] = normal_bits(seed, 1000 * (layer + 1) + 11, (T, filled, n_kv_heads, head_dim), 1.0, "f16")
    vc[:, :filled] = normal_bits(seed, 1000 * (layer + 1) + 12, (T, filled, n_kv_heads, head_dim), 1.0, "f16")
    return kc, vc


def hidden_state(seed: int, stream: int, T: int, hidden: int, scale: float = 1.0,
                 scales_stream: int | None = None) -> np.ndarray:
    """fp32 residual-stream input: Laplace draws times a persistent per-channel scale."""
    a = channel_scales(seed, scales_stream, hidden) if scales_stream is not None else 1.0
    return (laplace(seed, stream, (T, hidden), scale) * a).astype(np.float32)


# ---- device-side draws (bench-scale tensors: 13+ GB are drawn on the GPU in a second) ----

def device_normal_bits(seed: int, stream: int, shape, sigma: float, dtype: str):
    """N(0, sigma^2) rounded to dtype, drawn with torch's seeded CUDA generator.
    Returns an int16 CUDA tensor of bit patterns.  Input generation only."""
    import torch
    g = torch.Generator(device="cuda")
    g.manual_seed((int(seed) * 1000003 + int(stream)) & (2**63 - 1))
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=tdt, device="cuda")
    chunk = 1 << 26
    for o in range(0, n, chunk):
        m = min(chunk, n - o)
        out[o:o + m] = (torch.randn(m, generator=g, device="cuda", dtype=torch.float32) * sigma).to(tdt)
    return out.view(torch.int16).view(*shape)


def device_layer_weights(seed: int, layer: int, hidden: int, n_heads: int, n_kv_heads: int, mlp: int,
                         dtype: str, head_dim: int = 128, sigma: float = 0.02) -> dict:
    """Device-resident random-init layer (w_gu already in the interleaved gate/up layout:
    with i.i.d. entries any fixed column arrangement has the same distribution)."""
    import torch
    base = 1000 * (layer + 1)
    n_qkv = (n_heads + 2 * n_kv_heads) * head_dim
    return dict(
        w_qkv=device_normal_bits(seed, base + 1, (hidden, n_qkv), sigma, dtype),
        w_o=device_normal_bits(seed, base + 2, (n_heads * head_dim, hidden), sigma, dtype),
        w_gu=device_normal_bits(seed, base + 3, (hidden, 2 * mlp), sigma, dtype),
        w_down=device_normal_bits(seed, base + 5, (mlp, hidden), sigma, dtype),
        g_attn=torch.ones(hidden, dtype=torch.float32, device="cuda"),
        g_mlp=torch.ones(hidden, dtype=torch.float32, device="cuda"),
    )


def split_gate_up(w_gu: np.ndarray):
    """Inverse of interleave_gate_up: [K][2*mlp] -> (gate [K][mlp], up [K][mlp])."""
    K, N2 = w_gu.shape
    v = w_gu.reshape(K, N2 // 16, 2, 8)
    return (np.ascontiguousarray(v[:, :, 0, :]).reshape(K, N2 // 2),
            np.ascontiguousarray(v[:, :, 1, :]).reshape(K, N2 // 2))


# ---- 4-bit block-quantised weights (the storage type the paper evaluates) ----

def device_q4_weight(seed: int, stream: int, K: int, N: int, sigma: float = 0.02):
    """q4_weight's recipe drawn with torch's seeded CUDA generator: a uint8 CUDA tensor
    [K][q4_row_bytes(N)] (rounded normal codes, scales around 2.5 * sigma / 8 with either sign).
    Input generation only; not the same stream of numbers as q4_weight."""
    import torch
    g = torch.Generator(device="cuda")
    g.manual_seed((int(seed) * 1000003 + int(stream)) & (2**63 - 1))
    rows = torch.zeros((K, q4_row_bytes(N)), dtype=torch.uint8, device="cuda")
    step = max(1, (1 << 25) // N)
    for r0 in range(0, K, step):  # bounded temporaries
        r1 = min(K, r0 + step)
        q = torch.randn((r1 - r0, N // 32, 32), generator=g, device="cuda").mul_(8.0 / 2.5).add_(8.0).round_().clamp_(0, 15)
        q = q.to(torch.uint8)
        rows[r0:r1, : N // 2] = (q[:, :, :16] | (q[:, :, 16:] << 4)).reshape(r1 - r0, N // 2)
        d = sigma * 2.5 / 8.0 * (1.0 + 0.1 * torch.randn((r1 - r0, N // 32), generator=g, device="cuda"))
        d = d * (torch.rand((r1 - r0, N // 32), generator=g, device="cuda") < 0.5).to(torch.float32).mul_(2.0).sub_(1.0)
        rows[r0:r1, N // 2: N // 2 + N // 16] = d.to(torch.float16).view(torch.uint8)
    return rows


def q4_row_bytes(N: int) -> int:
    """Bytes of one channel of N outputs (N a multiple of 32) in the 4-bit layout: N/2 bytes of
    4-bit codes, then N/32 fp16 block scales, padded to a multiple of 16 bytes."""
    assert N % 32 == 0
    return (N // 2 + N // 16 + 15) // 16 * 16


def q4_weight(seed: int, stream: int, K: int, N: int, sigma: float = 0.02) -> np.ndarray:
    """Random-init channel-contiguous 4-bit weights, drawn directly in storage form: uint8
    [K][q4_row_bytes(N)].  Each block of 32 outputs has an fp16 scale d and 32 codes q in 0..15
    (value (q - 8) * d); codes are rounded normal draws with the spread a quantised N(0, sigma^2)
    block has (its largest magnitude lands near code 0 or 15), scales scatter around
    2.5 * sigma / 8.  Byte m of a block holds code m (low 4 bits) and code m + 16 (high 4 bits)."""
    g = rng(seed, stream)
    q = np.clip(np.rint(g.standard_normal((K, N // 32, 32), dtype=np.float32) * (8.0 / 2.5) + 8.0), 0, 15).astype(np.uint8)
    d = (sigma * 2.5 / 8.0 * (1.0 + 0.1 * g.standard_normal((K, N // 32), dtype=np.float32)))
    d *= np.where(g.random((K, N // 32)) < 0.5, -1.0, 1.0).astype(np.float32)   # the format allows negative scales
    rows = np.zeros((K, q4_row_bytes(N)), np.uint8)
    rows[:, : N // 2] = (q[:, :, :16] | (q[:, :, 16:] << 4)).reshape(K, N // 2)
    rows[:, N // 2: N // 2 + N // 16] = d.astype(np.float16).view(np.uint8).reshape(K, N // 16)
    return rows

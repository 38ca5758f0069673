"""Oracle composition of one Llama-shaped decoder layer with sparse operators (test
infrastructure; plain numpy over the C primitives of ``oracle``).

Structure after the paper's Fig. "simplified transformer layer structure" and Sec. 2.1
(every linear operator is evaluated on the active channels of its own input), cross-layer
prediction after Sec. 3.  The numerics the paper is silent about follow common Llama
practice: fp32-like residual carried here in fp64, every operator input rounded once to
the 16-bit storage type before selection, fp16 KV cache, rotary embedding on adjacent
pairs, softmax scale 1/sqrt(128).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

import oracle

OPS = ("qkv", "o", "gu", "down")


@dataclass
class LayerWeights:
    """uint16 bit patterns, channel-contiguous [K][N]; gains fp64."""
    w_qkv: np.ndarray   # [hidden][(Hq + 2 Hkv) * D]  columns q | k | v
    w_o: np.ndarray     # [Hq * D][hidden]
    w_gate: np.ndarray  # [hidden][mlp]
    w_up: np.ndarray    # [hidden][mlp]
    w_down: np.ndarray  # [mlp][hidden]
    g_attn: np.ndarray
    g_mlp: np.ndarray
    k: dict = field(default_factory=dict)    # op name -> top-k count
    tau: dict = field(default_factory=dict)  # op name -> threshold


@dataclass
class Config:
    dtype: str
    hidden: int
    n_heads: int
    n_kv_heads: int
    mlp: int
    head_dim: int = 128
    eps: float = 1e-5
    theta: float = 10000.0
    mode: int = oracle.TOPK
    xl_depth: int = 0
    xl_mode: int = 0     # 0 off, 1 bookkeeping (compute on the actual set), 2 reuse the predicted set


def select(x_bits, cfg: Config, lw: LayerWeights, op: str) -> np.ndarray:
    return oracle.select_active(x_bits, cfg.dtype, cfg.mode, k=lw.k.get(op, 0), tau=lw.tau.get(op, 0.0))


def attention_stage(cfg: Config, qkv, kc, vc, pos: int):
    """qkv fp64 [T][n_qkv]; kc, vc uint16 [T][max_seq][Hkv][D], row `pos` is written.
    Returns the attention output bits [T][Hq*D]."""
    T = qkv.shape[0]
    Hq, Hkv, D = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    out = np.empty((T, Hq * D), np.uint16)
    posv = np.full(1, pos, np.int32)
    for t in range(T):
        q = oracle.rope(qkv[t, : Hq * D].reshape(1, Hq, D), posv, cfg.theta)[0]
        k = oracle.rope(qkv[t, Hq * D:(Hq + Hkv) * D].reshape(1, Hkv, D), posv, cfg.theta)[0]
        v = qkv[t, (Hq + Hkv) * D:].reshape(Hkv, D)
        kc[t, pos] = oracle.round_to(k, "f16")
        vc[t, pos] = oracle.round_to(v, "f16")
        out[t] = oracle.attention(q, kc[t], vc[t], pos + 1, cfg.dtype).reshape(-1)
    return out


def mlp_block(cfg: Config, lw: LayerWeights, x_bits):
    """y = W_down(silu(W_gate x) * W_up x) on the active channels; x_bits [T][hidden]."""
    x_bits = np.atleast_2d(x_bits)
    a_gu = select(x_bits, cfg, lw, "gu")
    g = oracle.sparse_gemv(lw.w_gate, cfg.dtype, cfg.mlp, x_bits, a_gu)
    u = oracle.sparse_gemv(lw.w_up, cfg.dtype, cfg.mlp, x_bits, a_gu)
    hm = oracle.silu_mul(g, u, cfg.dtype)
    a_d = select(hm, cfg, lw, "down")
    y = oracle.sparse_gemv(lw.w_down, cfg.dtype, cfg.hidden, hm, a_d)
    return dict(idx_gu=a_gu, hm=hm, idx_down=a_d, y=y)


class CrossLayer:
    """Predicted sets per operator input (Sec. 3): layers p = 0, d, 2d, .. predict p+1 .. p+d."""

    def __init__(self, cfg: Config):
        self.cfg = cfg
        self.pred = {}

    def plan(self, layer: int):
        """(is_predictor, has_prediction)"""
        d = self.cfg.xl_depth
        if d <= 0 or self.cfg.xl_mode == 0:
            return False, False
        return layer % d == 0, layer > 0


def decoder_layer(cfg: Config, lw: LayerWeights, h, kc, vc, pos: int, layer: int = 0,
                  xl: CrossLayer | None = None):
    """One layer, free running.  h fp64 [T][hidden] -> dict with every intermediate."""
    h = np.atleast_2d(np.asarray(h, np.float64))
    rec = {}
    predictor, predicted = xl.plan(layer) if xl is not None else (False, False)

    def active(op, x_bits, K):
        reuse = predicted and not predictor and cfg.xl_mode == 2
        if reuse:
            idx = xl.pred[op]
        else:
            idx = select(x_bits, cfg, lw, op)
            if predicted:
                miss, hit = oracle.diff_active(idx, xl.pred[op], K)
                rec["miss_" + op], rec["hit_" + op] = miss, hit
            if predictor:
                rec["newpred_" + op] = idx
        rec["idx_" + op] = idx
        return idx

    xa = oracle.rmsnorm(h, lw.g_attn, cfg.eps, cfg.dtype)
    qkv = oracle.sparse_gemv(lw.w_qkv, cfg.dtype, lw.w_qkv.shape[1], xa, active("qkv", xa, cfg.hidden))
    attn = attention_stage(cfg, qkv, kc, vc, pos)
    h1 = h + oracle.sparse_gemv(lw.w_o, cfg.dtype, cfg.hidden, attn,
                                active("o", attn, cfg.n_heads * cfg.head_dim))
    xm = oracle.rmsnorm(h1, lw.g_mlp, cfg.eps, cfg.dtype)
    a_gu = active("gu", xm, cfg.hidden)
    g = oracle.sparse_gemv(lw.w_gate, cfg.dtype, cfg.mlp, xm, a_gu)
    u = oracle.sparse_gemv(lw.w_up, cfg.dtype, cfg.mlp, xm, a_gu)
    hm = oracle.silu_mul(g, u, cfg.dtype)
    h2 = h1 + oracle.sparse_gemv(lw.w_down, cfg.dtype, cfg.hidden, hm, active("down", hm, cfg.mlp))
    if xl is not None:
        for op in OPS:
            if "newpred_" + op in rec:
                xl.pred[op] = rec["newpred_" + op]
    rec.update(xnorm_qkv=xa, qkv=qkv, attn=attn, h1=h1, xnorm_gu=xm, hm=hm, h=h2)
    return rec


# ---- mixture-of-experts MLP (the Mixtral-shaped deployment of Sec. 1 / Sec. 7.2) ----

def moe_router(x_bits, w_router, dtype: str, top: int = 2):
    """Dense router of a sparse mixture-of-experts layer for ONE token: logits = W_r x over all
    channels (the router stays dense, only the experts' operators are sparse), the `top`
    experts by logit (equal logits: the lower expert id first), their weights the softmax over
    the chosen logits.  w_router: [hidden][E] bit patterns, channel-contiguous.
    Returns (expert ids in rank order, weights, logits)."""
    x = oracle.decode(np.asarray(x_bits, np.uint16).reshape(-1), dtype)
    W = oracle.decode(w_router, dtype)
    logits = np.zeros(W.shape[1])
    for j in range(W.shape[0]):          # ascending channel order, fp64
        logits += x[j] * W[j]
    order = sorted(range(W.shape[1]), key=lambda e: (-logits[e], e))[:top]
    z = np.exp(logits[order] - logits[order[0]])
    return np.array(order, np.int32), z / z.sum(), logits


def moe_block(cfg: Config, x_bits, w_router, experts, top: int = 2):
    """y = sum over the chosen experts of weight * W_down_e(silu(W_gate_e x) * W_up_e x), every
    expert operator on the active channels of its own input (mlp_block); experts: list of
    LayerWeights (only gate / up / down and their k / tau are used); one token."""
    ids, w, logits = moe_router(x_bits, w_router, cfg.dtype, top)
    y = np.zeros((1, cfg.hidden))
    parts = []
    for e, we in zip(ids, w):
        part = mlp_block(cfg, experts[int(e)], x_bits)
        parts.append(part)
        y = y + we * part["y"]
    return dict(experts=ids, weights=w, logits=logits, parts=parts, y=y)

"""Pins for the oracle's decoder-layer composition (oracle/layer.py), CPU only.

What fixes it from outside: (a) bookkeeping must not change a layer's output (Sec. 3: the
prediction only decides what is preloaded); (b) identical layers give identical operator
inputs, so nothing is missed and computing on the predicted set changes nothing; (c) the
group schedule written out by hand (who predicts whom, when a new prediction becomes
visible, the clipped last group); (d) a dense layer written here with plain numpy
(`@`, np.exp) that shares no code with the oracle; (e) a K = 8 case worked by hand.
"""
import math

import numpy as np
import pytest

import oracle
import oracle.layer as ol
from paper_2504_08378_b200 import synth

OPS = ol.OPS


def weights(L, k=None, tau=None):
    return ol.LayerWeights(L["w_qkv"], L["w_o"], L["w_gate"], L["w_up"], L["w_down"],
                           L["g_attn"].astype(np.float64), L["g_mlp"].astype(np.float64),
                           k=dict(zip(OPS, k or [0] * 4)), tau=dict(zip(OPS, tau or [0.0] * 4)))


def small_stack(seed, n_layers, dt, heads=2, kvh=1, mlp=384, same_layer=False, jitter=0.1):
    hidden = heads * 128
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    Ls = []
    for l in range(n_layers):
        L = synth.layer_weights(seed, 0 if same_layer else l, hidden, heads, kvh, mlp, dt, gain_jitter=jitter)
        Ls.append(L)
    return hidden, k, Ls


def run_stack(cfg, Ls, k, h0, pos, max_seq, seed, same_cache=False, xl=True):
    h = np.asarray(h0, np.float64)
    state = ol.CrossLayer(cfg) if xl else None
    recs = []
    for l, L in enumerate(Ls):
        kc, vc = synth.kv_cache(seed, 0 if same_cache else l, h.shape[0], max_seq, cfg.n_kv_heads, pos)
        rec = ol.decoder_layer(cfg, weights(L, k), h, kc, vc, pos, layer=l, xl=state)
        recs.append(rec)
        h = rec["h"]
    return recs


# ---- (a) bookkeeping never changes what a layer computes -----------------------------------

@pytest.mark.parametrize("dt", ["bf16", "f16"])
def test_bookkeeping_output_equals_plain_per_layer_selection(dt):
    hidden, k, Ls = small_stack(61, 7, dt)
    h0 = synth.hidden_state(61, 5, 1, hidden, scales_stream=6)
    plain = run_stack(ol.Config(dt, hidden, 2, 1, 384, mode=oracle.TOPK), Ls, k, h0, 9, 16, 61, xl=False)
    book = run_stack(ol.Config(dt, hidden, 2, 1, 384, mode=oracle.TOPK, xl_depth=3, xl_mode=1), Ls, k, h0, 9, 16, 61)
    for l in range(7):
        for name in ("xnorm_qkv", "qkv", "attn", "h1", "xnorm_gu", "hm", "h"):
            assert np.array_equal(plain[l][name], book[l][name]), (l, name)
        for op in OPS:
            assert np.array_equal(plain[l]["idx_" + op], book[l]["idx_" + op])
    # and the bookkeeping did happen: every layer after the first lists its misses
    assert all(("miss_" + op in book[l]) == (l > 0) for l in range(7) for op in OPS)
    assert any(book[l]["miss_qkv"].size > 0 for l in range(1, 7))


# ---- (b) identical layers: the prediction is perfect -----------------------------------------

@pytest.mark.parametrize("depth", [1, 3])
def test_identical_layers_with_silent_output_operators_miss_nothing(depth):
    dt = "bf16"
    hidden, k, Ls = small_stack(62, 6, dt, same_layer=True)
    for L in Ls:  # W_o = W_down = 0: the residual never changes, every layer sees the same inputs
        L["w_o"] = np.zeros_like(L["w_o"])
        L["w_down"] = np.zeros_like(L["w_down"])
    h0 = synth.hidden_state(62, 5, 1, hidden, scales_stream=6)
    out = {}
    for mode in (1, 2):
        cfg = ol.Config(dt, hidden, 2, 1, 384, mode=oracle.TOPK, xl_depth=depth, xl_mode=mode)
        out[mode] = run_stack(cfg, Ls, k, h0, 9, 16, 62, same_cache=True)
    for l in range(6):
        assert np.array_equal(out[1][l]["h"], h0.astype(np.float64))
        for i, op in enumerate(OPS):
            if l > 0:
                assert out[1][l]["miss_" + op].size == 0 and out[1][l]["hit_" + op] == k[i]
            assert np.array_equal(out[1][l]["idx_" + op], out[2][l]["idx_" + op])
        for name in ("qkv", "attn", "hm", "h"):
            assert np.array_equal(out[1][l][name], out[2][l][name]), (l, name)


# ---- (c) the schedule, against a table written by hand ----------------------------------------

# layer -> the layer whose sets it is compared with (None: nothing to compare with)
SCHEDULE = {
    3: {0: None, 1: 0, 2: 0, 3: 0, 4: 3, 5: 3, 6: 3, 7: 6},   # predictors 0, 3, 6; last group = {7}
    1: {0: None, 1: 0, 2: 1, 3: 2, 4: 3, 5: 4, 6: 5, 7: 6},   # every layer predicts the next one
}
PREDICTORS = {3: {0, 3, 6}, 1: set(range(8))}


@pytest.mark.parametrize("depth", [3, 1])
def test_bookkeeping_schedule_matches_hand_table(depth):
    dt = "f16"
    hidden, k, Ls = small_stack(63, 8, dt)
    h0 = synth.hidden_state(63, 5, 1, hidden, scale=4.0, scales_stream=6)
    cfg = ol.Config(dt, hidden, 2, 1, 384, mode=oracle.TOPK, xl_depth=depth, xl_mode=1)
    recs = run_stack(cfg, Ls, k, h0, 9, 16, 63)
    for l in range(8):
        p = SCHEDULE[depth][l]
        for op in OPS:
            A = recs[l]["idx_" + op]
            if p is None:
                assert "miss_" + op not in recs[l]
                continue
            P = recs[p]["idx_" + op]
            assert np.array_equal(recs[l]["miss_" + op], np.setdiff1d(A, P)), (l, op)
            assert recs[l]["hit_" + op] == np.intersect1d(A, P).size
            assert ("newpred_" + op in recs[l]) == (l in PREDICTORS[depth])
    # the inputs do differ from layer to layer, so a wrong predictor would have been seen
    assert any(not np.array_equal(recs[2]["idx_" + op], recs[1]["idx_" + op]) for op in OPS)
    assert recs[4]["miss_qkv"].size > 0


@pytest.mark.parametrize("depth", [3, 1])
def test_reuse_schedule_matches_hand_table(depth):
    """REUSE: a layer that is not a predictor computes on its predictor's sets and selects
    nothing; predictor layers (and layer 0) select for themselves."""
    dt = "bf16"
    hidden, k, Ls = small_stack(64, 8, dt)
    h0 = synth.hidden_state(64, 5, 1, hidden, scale=4.0, scales_stream=6)
    cfg = ol.Config(dt, hidden, 2, 1, 384, mode=oracle.TOPK, xl_depth=depth, xl_mode=2)
    recs = run_stack(cfg, Ls, k, h0, 9, 16, 64)
    inputs = {"qkv": "xnorm_qkv", "o": "attn", "gu": "xnorm_gu", "down": "hm"}
    for l in range(8):
        p = SCHEDULE[depth][l]
        for i, op in enumerate(OPS):
            own = oracle.select_active(recs[l][inputs[op]], dt, oracle.TOPK, k=k[i])
            if l in PREDICTORS[depth]:
                assert np.array_equal(recs[l]["idx_" + op], own), (l, op)
            else:
                assert np.array_equal(recs[l]["idx_" + op], recs[p]["idx_" + op]), (l, op)
    # computing on somebody else's set is visible in the result (depth 3 only: at depth 1
    # every layer is a predictor and REUSE never applies)
    if depth == 3:
        own = oracle.select_active(recs[1]["xnorm_qkv"], dt, oracle.TOPK, k=k[0])
        assert not np.array_equal(own, recs[1]["idx_qkv"])
        qkv_own = oracle.sparse_gemv(Ls[1]["w_qkv"], dt, Ls[1]["w_qkv"].shape[1], recs[1]["xnorm_qkv"], own)
        assert not np.array_equal(qkv_own, recs[1]["qkv"])
        qkv_pred = oracle.sparse_gemv(Ls[1]["w_qkv"], dt, Ls[1]["w_qkv"].shape[1], recs[1]["xnorm_qkv"],
                                      recs[0]["idx_qkv"])
        assert np.array_equal(qkv_pred, recs[1]["qkv"])


# ---- (d) an independent dense layer in plain numpy ---------------------------------------------

def np_decode(bits, dt):
    bits = np.asarray(bits, np.uint16)
    if dt == "f16":
        return bits.view(np.float16).astype(np.float64)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def np_round(v, dt):
    """One round-to-nearest-even from fp64 (normal range), independent of the oracle's."""
    v = np.asarray(v, np.float64)
    if dt == "f16":
        return v.astype(np.float16).view(np.uint16)
    m, e = np.frexp(v)                       # v = m * 2^e, 0.5 <= |m| < 1
    q = np.ldexp(np.rint(m * 256.0), e - 8)  # 8 significant bits, ties to even
    return (q.astype(np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def np_dense_layer(L, dt, h, kc, vc, pos, heads, kvh, eps=1e-5, theta=10000.0, D=128):
    """The layer with every operator dense, written from the Llama definition."""
    T, hidden = h.shape
    Wqkv, Wo = np_decode(L["w_qkv"], dt), np_decode(L["w_o"], dt)
    Wg, Wu, Wd = np_decode(L["w_gate"], dt), np_decode(L["w_up"], dt), np_decode(L["w_down"], dt)
    rep = heads // kvh
    out = {}
    xa = np_round(h / np.sqrt((h * h).mean(axis=1, keepdims=True) + eps) * L["g_attn"].astype(np.float64), dt)
    qkv = np_decode(xa, dt) @ Wqkv
    ang = pos * theta ** (-2.0 * np.arange(D // 2) / D)
    c, s = np.cos(ang), np.sin(ang)

    def rot(v):  # [heads][D], adjacent pairs
        a, b = v[:, 0::2], v[:, 1::2]
        r = np.empty_like(v)
        r[:, 0::2], r[:, 1::2] = a * c - b * s, a * s + b * c
        return r

    attn = np.empty((T, heads * D), np.uint16)
    kc, vc = kc.copy(), vc.copy()
    for t in range(T):
        q = rot(qkv[t, :heads * D].reshape(heads, D))
        kk = rot(qkv[t, heads * D:(heads + kvh) * D].reshape(kvh, D))
        vv = qkv[t, (heads + kvh) * D:].reshape(kvh, D)
        kc[t, pos] = kk.astype(np.float16).view(np.uint16)
        vc[t, pos] = vv.astype(np.float16).view(np.uint16)
        Kf = kc[t, :pos + 1].view(np.float16).astype(np.float64)  # [L][kvh][D]
        Vf = vc[t, :pos + 1].view(np.float16).astype(np.float64)
        o = np.empty((heads, D))
        for hq in range(heads):
            sc = Kf[:, hq // rep, :] @ q[hq] / math.sqrt(D)
            p = np.exp(sc - sc.max())
            o[hq] = (p / p.sum()) @ Vf[:, hq // rep, :]
        attn[t] = np_round(o.reshape(-1), dt)
    h1 = h + np_decode(attn, dt) @ Wo
    xm = np_round(h1 / np.sqrt((h1 * h1).mean(axis=1, keepdims=True) + eps) * L["g_mlp"].astype(np.float64), dt)
    g, u = np_decode(xm, dt) @ Wg, np_decode(xm, dt) @ Wu
    hm = np_round(g / (1.0 + np.exp(-g)) * u, dt)
    h2 = h1 + np_decode(hm, dt) @ Wd
    out.update(xnorm_qkv=xa, qkv=qkv, attn=attn, h1=h1, xnorm_gu=xm, hm=hm, h=h2, kc=kc, vc=vc)
    return out


@pytest.mark.parametrize("dt,heads,kvh,T", [("bf16", 4, 2, 1), ("f16", 4, 4, 1), ("bf16", 4, 1, 3)])
def test_layer_without_sparsity_equals_plain_numpy_dense_layer(dt, heads, kvh, T):
    hidden, mlp, pos, max_seq = heads * 128, 328, 11, 14
    L = synth.layer_weights(65, 0, hidden, heads, kvh, mlp, dt, gain_jitter=0.2)
    h0 = synth.hidden_state(65, 5, T, hidden, scales_stream=6).astype(np.float64)
    kc, vc = synth.kv_cache(65, 0, T, max_seq, kvh, pos)
    ref = np_dense_layer(L, dt, h0, kc, vc, pos, heads, kvh)
    K_op = [hidden, heads * 128, hidden, mlp]
    variants = [ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK),       # k = K keeps everything
                ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.THRESHOLD)]  # tau < 0 keeps everything
    for cfg in variants:
        kco, vco = kc.copy(), vc.copy()
        rec = ol.decoder_layer(cfg, weights(L, K_op, [-1.0] * 4), h0, kco, vco, pos)
        for name in ("xnorm_qkv", "attn", "xnorm_gu", "hm"):
            assert np.array_equal(rec[name], ref[name]), name
        assert np.array_equal(kco, ref["kc"]) and np.array_equal(vco, ref["vc"])
        scale = np.abs(ref["h"]).max()
        for name in ("qkv", "h1", "h"):
            assert np.abs(rec[name] - ref[name]).max() <= 1e-12 * max(scale, 1.0), name
        for i, op in enumerate(OPS):
            assert np.array_equal(rec["idx_" + op], np.arange(K_op[i]))


# ---- (e) K = 8 by hand, through mlp_block ----------------------------------------------------

def test_mlp_block_hand_case():
    """x = [0.5, -2, 1, -1, 0, 3, -3, 0.25], top 4 of |x| = {1, 2, 5, 6} (the tie 1 = |-1| goes
    to channel 2).  Gate and up are the identity, so hm_j = silu(x_j) * x_j on those four
    channels and 0 elsewhere; the top 2 of |hm| are channels 5 and 2; W_down's rows are
    r[j] = (j + 1, +-1, 0, ...), so y = hm_2 * r[2] + hm_5 * r[5]."""
    dt = "f16"
    x = np.array([0.5, -2, 1, -1, 0, 3, -3, 0.25], np.float32)
    xb = synth.f32_to_bits(x, dt)[None, :]
    eye = synth.f32_to_bits(np.eye(8, dtype=np.float32), dt)
    wd = np.zeros((8, 8), np.float32)
    wd[:, 0] = np.arange(1, 9)
    wd[:, 1] = [1, -1, 1, -1, 1, -1, 1, -1]
    cfg = ol.Config(dt, 8, 1, 1, 8, mode=oracle.TOPK)
    lw = ol.LayerWeights(None, None, eye, eye, synth.f32_to_bits(wd, dt), None, None, k={"gu": 4, "down": 2})
    out = ol.mlp_block(cfg, lw, xb)
    assert out["idx_gu"].tolist() == [1, 2, 5, 6]
    hm = np.zeros(8)
    for j in (1, 2, 5, 6):
        v = float(x[j])
        hm[j] = float(np.float16(v / (1.0 + math.exp(-v)) * v))  # 0.4768, 0.7310, 8.57, 0.4268
    assert np.array_equal(out["hm"][0], np.array(hm, np.float16).view(np.uint16))
    assert out["idx_down"].tolist() == [2, 5]
    y = np.zeros(8)
    y[0] = hm[2] * 3 + hm[5] * 6
    y[1] = hm[2] * 1 + hm[5] * -1
    assert np.allclose(out["y"][0], y, rtol=0, atol=1e-12)
    # by pocket calculator: hm_2 = 0.73096, hm_5 = 8.5703 (fp16 steps of 2^-7 there)
    assert abs(out["y"][0][0] - 53.615) < 0.002 and abs(out["y"][0][1] + 7.8394) < 0.002


def test_attention_stage_appends_at_pos_and_maps_grouped_heads():
    """Row `pos` of the caches receives the rotated k and the plain v of the current token
    (fp16), rows before it stay, and query head h reads kv head h // (Hq / Hkv)."""
    dt, Hq, Hkv, D, pos = "bf16", 4, 2, 128, 3
    cfg = ol.Config(dt, Hq * D, Hq, Hkv, 64)
    g = synth.rng(66, 1)
    qkv = g.standard_normal((1, (Hq + 2 * Hkv) * D))
    kc, vc = synth.kv_cache(66, 0, 1, 6, Hkv, pos)
    kc0, vc0 = kc.copy(), vc.copy()
    out = ol.attention_stage(cfg, qkv, kc, vc, pos)
    assert np.array_equal(kc[:, :pos], kc0[:, :pos]) and np.array_equal(vc[:, :pos], vc0[:, :pos])
    assert np.array_equal(kc[:, pos + 1:], kc0[:, pos + 1:])
    v_now = qkv[0, (Hq + Hkv) * D:].reshape(Hkv, D)
    assert np.array_equal(vc[0, pos], v_now.astype(np.float16).view(np.uint16))
    k_now = qkv[0, Hq * D:(Hq + Hkv) * D].reshape(Hkv, D)
    ang = pos * 10000.0 ** (-2.0 * np.arange(D // 2) / D)
    kr = np.empty_like(k_now)
    kr[:, 0::2] = k_now[:, 0::2] * np.cos(ang) - k_now[:, 1::2] * np.sin(ang)
    kr[:, 1::2] = k_now[:, 0::2] * np.sin(ang) + k_now[:, 1::2] * np.cos(ang)
    assert np.array_equal(kc[0, pos], kr.astype(np.float16).view(np.uint16))
    # zero the values of kv head 1: exactly the query heads 2 and 3 must go to zero
    vc2 = vc.copy()
    vc2[:, :, 1, :] = 0
    qkv2 = qkv.copy()
    qkv2[0, (Hq + Hkv) * D + D:] = 0.0
    out2 = ol.attention_stage(cfg, qkv2, kc.copy(), vc2, pos).reshape(Hq, D)
    assert np.array_equal(out2[:2], out.reshape(Hq, D)[:2]) and not out2[2:].any()

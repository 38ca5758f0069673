"""GPU parity for the fused decoder-layer kernels, one operator at a time: each stage's
output is checked against the oracle run on the SAME stage input the GPU recorded."""
import numpy as np
import pytest
import torch

import oracle
import oracle.layer as ol
from paper_2504_08378_b200 import afx, synth
from paper_2504_08378_b200.model import DecoderModel
from gpu_util import rel_err

pytestmark = pytest.mark.gpu

TOL = 2e-3
OPN = ["qkv", "o", "gu", "down"]


def bits_np(t):
    return t.cpu().numpy().view(np.uint16)


EPS32 = 2.0 ** -24
# Longest chain of fp32 additions behind one output of the sparse GEMV kernels at the shapes
# tested: at most 48 channels per accumulator, 16 warps, 8 blocks of a cluster, the lane-group
# shuffles and the residual add.  |fp32 sum - exact sum| <= SUM_DEPTH * EPS32 * sum |terms|.
SUM_DEPTH = 96


def ulp_close(a, b, frac_exact=0.98, dt=None, abs_err=None):
    """16-bit results of the same arithmetic in fp32 (GPU, `a`) and fp64 (oracle, `b`): nearly
    all bit patterns equal, the rest one step apart.  Where a value comes out of a sum that
    cancels, one step of the 16-bit type can be far below the fp32 sum's own rounding error;
    `abs_err` (same shape, needs dt) is the bound on that error carried to the value before
    its final rounding, and an element passes if it is within abs_err + one step."""
    d = np.abs(a.astype(np.int32) - b.astype(np.int32))
    ok = d <= 1
    if abs_err is not None and not ok.all():
        va, vb = oracle.decode(a, dt), oracle.decode(b, dt)
        step = np.abs(vb) * 2.0 ** (-7 if dt == "bf16" else -10) + 2.0 ** (-133 if dt == "bf16" else -24)
        ok |= np.abs(va - vb) <= abs_err + step
    return ok.all() and (d == 0).mean() >= frac_exact


def abs_gemv(W_bits, dt, x_bits, idx):
    """sum_c |x[t][idx[c]]| * |W[idx[c]][i]|: the magnitude scale of a sparse GEMV's rounding error."""
    return np.abs(oracle.decode(np.atleast_2d(x_bits)[:, idx], dt)) @ np.abs(oracle.decode(W_bits[idx], dt))


def silu_mul_err(g, u, abs_g, abs_u):
    """Bound on |silu(g') u' - silu(g) u| for |g' - g| <= SUM_DEPTH*EPS32*abs_g (same for u):
    |silu'| <= 1.1 everywhere; plus a few fp32 roundings of the product itself."""
    eg, eu = SUM_DEPTH * EPS32 * abs_g, SUM_DEPTH * EPS32 * abs_u
    sg = np.abs(g / (1.0 + np.exp(-g)))
    return 1.1 * (np.abs(u) + eu) * eg + sg * eu + 8 * EPS32 * sg * np.abs(u)


def make(cfg, layers_np, T, mode, xl_depth=0, xl_mode=0, max_seq=64):
    return DecoderModel(cfg.dtype, cfg.hidden, cfg.n_heads, cfg.n_kv_heads, cfg.mlp, max_seq, layers_np, T=T,
                        select_mode=mode, xl_depth=xl_depth, xl_mode=xl_mode)


def oracle_weights(L, k=None, tau=None):
    return ol.LayerWeights(L["w_qkv"], L["w_o"], L["w_gate"], L["w_up"], L["w_down"],
                           L["g_attn"].astype(np.float64), L["g_mlp"].astype(np.float64),
                           k=dict(zip(OPN, k or [0] * 4)), tau=dict(zip(OPN, tau or [0.0] * 4)))


def check_layer_stages(cfg, L, lw, m, layer, h0, kc0, vc0, pos, T, lists=None):
    """Teacher-forced comparison of every stage of one layer step already run on the GPU.
    `lists` (operator name -> index list) replaces the layer's own selection where the layer
    is expected to compute on somebody else's set (cross-layer REUSE)."""
    dt = cfg.dtype

    def expected(op, x_bits):
        return lists[op] if lists is not None else ol.select(x_bits, cfg, lw, op)

    Hq, Hkv, D = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    stats = m.stats.cpu().numpy()[layer]
    # qkv: norm -> select -> GEMV
    xa_gpu = bits_np(m.bits(afx.BUF_XNORM, afx.OP_QKV))
    xa_ref = oracle.rmsnorm(h0.astype(np.float64), lw.g_attn, cfg.eps, dt)
    assert ulp_close(xa_gpu, xa_ref)
    idx = m.idx(afx.OP_QKV).cpu().numpy()[: stats[0][0]]
    assert np.array_equal(idx, expected("qkv", xa_gpu))
    qkv_gpu = m.qkv.cpu().numpy()
    qkv_ref = oracle.sparse_gemv(L["w_qkv"], dt, L["w_qkv"].shape[1], xa_gpu, idx)
    assert rel_err(qkv_gpu, qkv_ref) <= TOL
    # attention on the GPU's own q, k, v
    kc, vc = kc0.copy(), vc0.copy()
    attn_ref = ol.attention_stage(cfg, qkv_gpu.astype(np.float64), kc, vc, pos)
    attn_gpu = bits_np(m.bits(afx.BUF_ATTN))
    kc_gpu = bits_np(m.k_cache[layer])
    vc_gpu = bits_np(m.v_cache[layer])
    assert ulp_close(kc_gpu[:, pos], kc[:, pos]) and ulp_close(vc_gpu[:, pos], vc[:, pos])
    assert np.array_equal(kc_gpu[:, :pos], kc0[:, :pos]), "past cache rows must not change"
    a_gpu, a_ref = oracle.decode(attn_gpu, dt), oracle.decode(attn_ref, dt)
    assert rel_err(a_gpu, a_ref) <= 2 * 2.0 ** (-8 if dt == "bf16" else -11) + 1e-3
    # o
    idx_o = m.idx(afx.OP_O).cpu().numpy()[: stats[1][0]]
    assert np.array_equal(idx_o, expected("o", attn_gpu))
    h1_ref = h0.astype(np.float64) + oracle.sparse_gemv(L["w_o"], dt, cfg.hidden, attn_gpu, idx_o)
    # gate/up
    xm_gpu = bits_np(m.bits(afx.BUF_XNORM, afx.OP_GU))
    # error of h1 = h + W_o a in fp32, carried through the normalisation (scale inv * gain)
    inv = 1.0 / np.sqrt((h1_ref ** 2).mean(axis=1, keepdims=True) + cfg.eps)
    h1_err = SUM_DEPTH * EPS32 * (np.abs(h0) + abs_gemv(L["w_o"], dt, attn_gpu, idx_o))
    xm_err = (h1_err + 8 * EPS32 * np.abs(h1_ref)) * inv * np.abs(lw.g_mlp)
    assert ulp_close(xm_gpu, oracle.rmsnorm(h1_ref, lw.g_mlp, cfg.eps, dt), frac_exact=0.97, dt=dt, abs_err=xm_err)
    idx_gu = m.idx(afx.OP_GU).cpu().numpy()[: stats[2][0]]
    assert np.array_equal(idx_gu, expected("gu", xm_gpu))
    g = oracle.sparse_gemv(L["w_gate"], dt, cfg.mlp, xm_gpu, idx_gu)
    u = oracle.sparse_gemv(L["w_up"], dt, cfg.mlp, xm_gpu, idx_gu)
    hm_gpu = bits_np(m.bits(afx.BUF_HM))
    hm_err = silu_mul_err(g, u, abs_gemv(L["w_gate"], dt, xm_gpu, idx_gu), abs_gemv(L["w_up"], dt, xm_gpu, idx_gu))
    assert ulp_close(hm_gpu, oracle.silu_mul(g, u, dt), frac_exact=0.97, dt=dt, abs_err=hm_err)
    # down
    idx_d = m.idx(afx.OP_DOWN).cpu().numpy()[: stats[3][0]]
    assert np.array_equal(idx_d, expected("down", hm_gpu))
    h2_ref = h1_ref + oracle.sparse_gemv(L["w_down"], dt, cfg.hidden, hm_gpu, idx_d)
    assert rel_err(m.h.cpu().numpy(), h2_ref) <= TOL
    return dict(idx=[idx, idx_o, idx_gu, idx_d], stats=stats,
                inputs=[xa_gpu, attn_gpu, xm_gpu, hm_gpu], kc=kc_gpu, vc=vc_gpu)


@pytest.mark.parametrize("dt", ["bf16", "f16"])
@pytest.mark.parametrize("T,mode,heads,kvh", [(1, afx.MODE_TOPK, 4, 4), (1, afx.MODE_THRESHOLD, 8, 2),
                                              (4, afx.MODE_TOPK, 4, 4), (8, afx.MODE_TOPK, 4, 2)])
def test_layer_step_every_stage_matches_oracle(dt, T, mode, heads, kvh):
    hidden, mlp, max_seq, pos = heads * 128, 1384, 48, 37
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=mode)
    L = synth.layer_weights(31, 0, hidden, heads, kvh, mlp, dt, gain_jitter=0.1)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    tau = [0.6, 0.02, 0.6, 0.004]
    L["k"], L["tau"] = k, tau
    kc0, vc0 = synth.kv_cache(31, 0, T, max_seq, kvh, pos)
    L["k_cache"], L["v_cache"] = kc0, vc0
    h0 = synth.hidden_state(31, 5, T, hidden, scales_stream=6)
    m = make(cfg, [L], T, mode, max_seq=max_seq)
    m.h.copy_(torch.from_numpy(h0).cuda())
    m.layer_step(0, pos)
    torch.cuda.synchronize()
    out = check_layer_stages(cfg, L, oracle_weights(L, k, tau), m, 0, h0, kc0, vc0, pos, T)
    if mode == afx.MODE_TOPK and T == 1:
        assert [len(i) for i in out["idx"]] == k
    m.close()


@pytest.mark.parametrize("xl_mode", [afx.XL_BOOKKEEP, afx.XL_REUSE])
def test_cross_layer_prediction_matches_oracle_free_running(xl_mode):
    """Four layers, depth 3: free-running GPU vs free-running oracle.  Index sets are compared
    exactly; a rare rounding flip at a top-k boundary would show up here as a set difference."""
    dt, heads, kvh, mlp, T, max_seq, pos, depth = "bf16", 4, 4, 1024, 1, 32, 20, 3
    hidden = heads * 128
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK, xl_depth=depth, xl_mode=xl_mode)
    layers, lws, caches = [], [], []
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    for l in range(4):
        L = synth.layer_weights(41, l, hidden, heads, kvh, mlp, dt)
        L["k"] = k
        kc0, vc0 = synth.kv_cache(41, l, T, max_seq, kvh, pos)
        L["k_cache"], L["v_cache"] = kc0, vc0
        layers.append(L)
        lws.append(oracle_weights(L, k))
        caches.append((kc0.copy(), vc0.copy()))
    h0 = synth.hidden_state(41, 5, T, hidden, scale=4.0, scales_stream=6)
    m = make(cfg, layers, T, afx.MODE_TOPK, xl_depth=depth, xl_mode=xl_mode, max_seq=max_seq)
    m.h.copy_(torch.from_numpy(h0).cuda())
    xl = ol.CrossLayer(cfg)
    h = h0.astype(np.float64)
    for l in range(4):
        m.layer_step(l, pos)
        torch.cuda.synchronize()
        rec = ol.decoder_layer(cfg, lws[l], h, caches[l][0], caches[l][1], pos, layer=l, xl=xl)
        h = rec["h"]
        stats = m.stats.cpu().numpy()[l]
        for op, name in enumerate(OPN):
            want = rec["idx_" + name]
            got = m.idx(op).cpu().numpy()[: stats[op][0]]
            assert np.array_equal(got, want), (l, name)
            if "miss_" + name in rec:
                assert stats[op][1] == rec["hit_" + name] and stats[op][2] == rec["miss_" + name].size
                assert np.array_equal(m.miss(op).cpu().numpy()[: stats[op][2]], rec["miss_" + name])
        assert rel_err(m.h.cpu().numpy(), h) <= TOL
    m.close()


def hm_close(L, dt, mlp, x_bits, idx_gu, hm_gpu, hm_ref, frac_exact=0.97):
    """silu(gate)*up of the GPU against the oracle's, with the fp32 sums' error bound."""
    g = oracle.sparse_gemv(L["w_gate"], dt, mlp, x_bits, idx_gu)
    u = oracle.sparse_gemv(L["w_up"], dt, mlp, x_bits, idx_gu)
    err = silu_mul_err(g, u, abs_gemv(L["w_gate"], dt, x_bits, idx_gu), abs_gemv(L["w_up"], dt, x_bits, idx_gu))
    return ulp_close(hm_gpu, hm_ref, frac_exact=frac_exact, dt=dt, abs_err=err)


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_mlp_block_threshold_sweep(dt):
    hidden, mlp, T = 1024, 2752, 1
    cfg = ol.Config(dt, hidden, 8, 8, mlp, mode=oracle.THRESHOLD)
    L = synth.layer_weights(51, 0, hidden, 8, 8, mlp, dt)
    x = synth.laplace_bits(51, 9, (T, hidden), dt)
    for p, tau_d in ((0.0, -1.0), (0.5, 0.004), (0.9, 0.02)):
        tau = [0.0, 0.0, synth.laplace_tau(p), tau_d]
        L["tau"] = tau
        m = make(cfg, [L], T, afx.MODE_THRESHOLD)
        xd = torch.from_numpy(x.view(np.int16)).cuda()
        y = torch.full((T, hidden), float("nan"), device="cuda")
        m.mlp_block(0, xd, y)
        torch.cuda.synchronize()
        ref = ol.mlp_block(cfg, oracle_weights(L, None, tau), x)
        stats = m.stats.cpu().numpy()[0]
        assert np.array_equal(m.idx(afx.OP_GU).cpu().numpy()[: stats[2][0]], ref["idx_gu"])
        hm_gpu = bits_np(m.bits(afx.BUF_HM))
        assert hm_close(L, dt, mlp, x, ref["idx_gu"], hm_gpu, ref["hm"])
        idx_d = m.idx(afx.OP_DOWN).cpu().numpy()[: stats[3][0]]
        assert np.array_equal(idx_d, oracle.select_active(hm_gpu, dt, oracle.THRESHOLD, tau=tau_d))
        y_ref = oracle.sparse_gemv(L["w_down"], dt, hidden, hm_gpu, idx_d)
        assert rel_err(y.cpu().numpy(), y_ref) <= TOL
        m.close()


def kth_key(bits, k):
    keys = np.sort(bits.reshape(-1).astype(np.int64) & 0x7FFF)
    return int(keys[keys.size - k])


@pytest.mark.parametrize("ties", [False, True])
@pytest.mark.parametrize("dt", ["bf16", "f16"])
def test_topk_search_hint_never_changes_the_selection(dt, ties):
    """Each one-token top-k selection records its k-th key; the next token's search starts in
    a window around it.  Whatever that hint is -- exact, a few keys off, at the window's
    edges, far outside, the extremes, absent -- every stage still matches the oracle, with
    many equal magnitudes at the boundary too."""
    heads, kvh, T, max_seq, pos = 4, 4, 1, 48, 37
    hidden, mlp = heads * 128, 1384
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK)
    L = synth.layer_weights(33, 0, hidden, heads, kvh, mlp, dt, gain_jitter=0.0 if ties else 0.1)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    L["k"] = k
    kc0, vc0 = synth.kv_cache(33, 0, T, max_seq, kvh, pos)
    L["k_cache"], L["v_cache"] = kc0, vc0
    h0 = synth.hidden_state(33, 5, T, hidden)
    if ties:
        h0 = np.round(h0 * 1.5).astype(np.float32)  # a handful of distinct magnitudes
    lw = oracle_weights(L, k)
    m = make(cfg, [L], T, afx.MODE_TOPK, max_seq=max_seq)
    half = 32 if dt == "bf16" else 256

    def run(hints):
        m.h.copy_(torch.from_numpy(h0).cuda())
        if hints is not None:
            m.stats[0, :, 3] = torch.tensor(hints, dtype=torch.int32, device="cuda")
        m.layer_step(0, pos)
        torch.cuda.synchronize()
        out = check_layer_stages(cfg, L, lw, m, 0, h0, kc0, vc0, pos, T)
        assert [len(i) for i in out["idx"]] == k
        return out

    run(None)  # state just created: no hint
    inputs = [bits_np(m.bits(afx.BUF_XNORM, afx.OP_QKV)), bits_np(m.bits(afx.BUF_ATTN)),
              bits_np(m.bits(afx.BUF_XNORM, afx.OP_GU)), bits_np(m.bits(afx.BUF_HM))]
    exact = [kth_key(b, kk) for b, kk in zip(inputs, k)]
    assert m.stats.cpu().numpy()[0, :, 3].tolist() == [0x10000 | e for e in exact]
    clamp = lambda v: min(0x7FFF, max(0, v))
    for delta in (0, 1, -1, 7, half - 1, -half, half, -half - 1, 5 * half, -5 * half):
        out = run([0x10000 | clamp(e + delta) for e in exact])
        assert out["stats"][:, 3].tolist() == [0x10000 | e for e in exact], delta
    for raw in (0x10000, 0x10000 | 0x7FFF, 0, 0x7FFF, -1):
        out = run([raw] * 4)
        assert out["stats"][:, 3].tolist() == [0x10000 | e for e in exact], raw
    m.close()


@pytest.mark.parametrize("dt", ["bf16", "f16"])
@pytest.mark.parametrize("T", [2, 4, 8])
def test_per_token_search_hints_never_change_the_selection(dt, T):
    """Several tokens per step: each token's top-k search starts from the k-th key its slot
    recorded last time.  First step without hints, then with its own keys as hints, then with
    hints that are off by a few keys, at the window's edge, far away, and garbage: every stage
    still matches the oracle, and the recorded keys are the exact k-th keys of each token."""
    heads, kvh, max_seq, pos = 4, 2, 48, 37
    hidden, mlp = heads * 128, 1384
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK)
    L = synth.layer_weights(35, 0, hidden, heads, kvh, mlp, dt, gain_jitter=0.1)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    L["k"] = k
    kc0, vc0 = synth.kv_cache(35, 0, T, max_seq, kvh, pos)
    L["k_cache"], L["v_cache"] = kc0, vc0
    h0 = synth.hidden_state(35, 5, T, hidden)
    lw = oracle_weights(L, k)
    m = make(cfg, [L], T, afx.MODE_TOPK, max_seq=max_seq)
    half = 32 if dt == "bf16" else 256

    def run(hints):
        m.h.copy_(torch.from_numpy(h0).cuda())
        if hints is not None:
            m.hints[0, :, :T] = torch.tensor(hints, dtype=torch.int32, device="cuda")
        m.layer_step(0, pos)
        torch.cuda.synchronize()
        return check_layer_stages(cfg, L, lw, m, 0, h0, kc0, vc0, pos, T)

    out = run(None)
    exact = [[kth_key(out["inputs"][op][t], k[op]) for t in range(T)] for op in range(4)]
    want = [[0x10000 | e for e in row] for row in exact]
    assert m.hints.cpu().numpy()[0, :, :T].tolist() == want
    clamp = lambda v: min(0x7FFF, max(0, v))
    for delta in (0, 3, -half, half, 7 * half):
        run([[0x10000 | clamp(e + delta * (1 if t % 2 else -1)) for t, e in enumerate(row)] for row in exact])
        assert m.hints.cpu().numpy()[0, :, :T].tolist() == want, delta
    for raw in (0, 0x10000, 0x10000 | 0x7FFF, -1):
        run([[raw] * T] * 4)
        assert m.hints.cpu().numpy()[0, :, :T].tolist() == want, raw
    m.close()

"""GPU parity for the decoder-layer step over 4-bit weights (afx_layer_step_q4): every stage
against the oracle run on the stage input the GPU recorded.  The input stage, the selection and
the attention are the kernels of the 16-bit step; the operators read channel-contiguous 4-bit
rows, and gate|up keeps 16 gate and 16 up outputs in every block of 32."""
import numpy as np
import pytest
import torch

import oracle
import oracle.layer as ol
from paper_2504_08378_b200 import afx, synth
from gpu_util import rel_err
from test_gpu_layer import EPS32, OPN, SUM_DEPTH, TOL, bits_np, make, oracle_weights, silu_mul_err, ulp_close

pytestmark = pytest.mark.gpu


def q4_layer_weights(seed, layer, hidden, n_attn, n_qkv, mlp, sigma=0.02):
    """uint8 rows per operator: q|k|v [hidden][.], o [n_attn][.], gate|up [hidden][.], down [mlp][.]."""
    base = 7000 + 10 * layer
    return [synth.q4_weight(seed, base + 1, hidden, n_qkv, sigma), synth.q4_weight(seed, base + 2, n_attn, hidden, sigma),
            synth.q4_weight(seed, base + 3, hidden, 2 * mlp, sigma), synth.q4_weight(seed, base + 4, mlp, hidden, sigma)]


def q4_struct(dev_rows, use=(True, True, True, True)):
    q = afx.Q4Layer()
    for op in range(4):
        q.wq[op] = dev_rows[op].data_ptr() if use[op] else None
        q.ldq_bytes[op] = dev_rows[op].shape[1] if use[op] else 0
    return q


def abs_gemv_q4(rows, N, dt, x_bits, idx):
    return np.abs(oracle.decode(np.atleast_2d(x_bits)[:, idx], dt)) @ np.abs(oracle.q4_decode(rows[idx], N))


def gate_up(y):
    """[1][N] outputs of the 4-bit gate|up rows -> (gate [1][N/2], up [1][N/2])."""
    b = y.reshape(y.shape[0], -1, 32)
    return b[:, :, :16].reshape(y.shape[0], -1), b[:, :, 16:].reshape(y.shape[0], -1)


def check_q4_stages(cfg, L16, q4rows, use, lw, m, layer, h0, kc0, vc0, pos, lists=None):
    """`lists` (operator name -> index list): the sets the layer must have computed on when it
    reuses another layer's (cross-layer REUSE)."""
    dt = cfg.dtype

    def expected(op, x_bits):
        return lists[op] if lists is not None else ol.select(x_bits, cfg, lw, op)

    stats = m.stats.cpu().numpy()[layer]
    n_qkv = (cfg.n_heads + 2 * cfg.n_kv_heads) * cfg.head_dim

    def gemv(op, N, x_bits, idx, w16):
        if use[op]:
            return oracle.sparse_gemv_q4(q4rows[op], N, x_bits, dt, idx)
        return oracle.sparse_gemv(w16, dt, N, x_bits, idx)

    # q|k|v
    xa_gpu = bits_np(m.bits(afx.BUF_XNORM, afx.OP_QKV))
    assert ulp_close(xa_gpu, oracle.rmsnorm(h0.astype(np.float64), lw.g_attn, cfg.eps, dt))
    idx = m.idx(afx.OP_QKV).cpu().numpy()[: stats[0][0]]
    assert np.array_equal(idx, expected("qkv", xa_gpu))
    qkv_gpu = m.qkv.cpu().numpy()
    assert rel_err(qkv_gpu, gemv(0, n_qkv, xa_gpu, idx, L16["w_qkv"])) <= TOL
    # attention on the GPU's own q, k, v
    kc, vc = kc0.copy(), vc0.copy()
    attn_ref = ol.attention_stage(cfg, qkv_gpu.astype(np.float64), kc, vc, pos)
    attn_gpu = bits_np(m.bits(afx.BUF_ATTN))
    assert rel_err(oracle.decode(attn_gpu, dt), oracle.decode(attn_ref, dt)) <= 2 * 2.0 ** (-8 if dt == "bf16" else -11) + 1e-3
    # o
    idx_o = m.idx(afx.OP_O).cpu().numpy()[: stats[1][0]]
    assert np.array_equal(idx_o, expected("o", attn_gpu))
    h1_ref = h0.astype(np.float64) + gemv(1, cfg.hidden, attn_gpu, idx_o, L16["w_o"])
    # gate|up: the normalised input carries the fp32 error of h + W_o a
    xm_gpu = bits_np(m.bits(afx.BUF_XNORM, afx.OP_GU))
    inv = 1.0 / np.sqrt((h1_ref ** 2).mean(axis=1, keepdims=True) + cfg.eps)
    if use[1]:
        abs_o = abs_gemv_q4(q4rows[1], cfg.hidden, dt, attn_gpu, idx_o)
    else:
        abs_o = np.abs(oracle.decode(attn_gpu[:, idx_o], dt)) @ np.abs(oracle.decode(L16["w_o"][idx_o], dt))
    h1_err = SUM_DEPTH * EPS32 * (np.abs(h0) + abs_o)
    xm_err = (h1_err + 8 * EPS32 * np.abs(h1_ref)) * inv * np.abs(lw.g_mlp)
    assert ulp_close(xm_gpu, oracle.rmsnorm(h1_ref, lw.g_mlp, cfg.eps, dt), frac_exact=0.97, dt=dt, abs_err=xm_err)
    idx_gu = m.idx(afx.OP_GU).cpu().numpy()[: stats[2][0]]
    assert np.array_equal(idx_gu, expected("gu", xm_gpu))
    hm_gpu = bits_np(m.bits(afx.BUF_HM))
    if use[2]:
        g, u = gate_up(oracle.sparse_gemv_q4(q4rows[2], 2 * cfg.mlp, xm_gpu, dt, idx_gu))
        ag, au = gate_up(abs_gemv_q4(q4rows[2], 2 * cfg.mlp, dt, xm_gpu, idx_gu))
    else:
        g = oracle.sparse_gemv(L16["w_gate"], dt, cfg.mlp, xm_gpu, idx_gu)
        u = oracle.sparse_gemv(L16["w_up"], dt, cfg.mlp, xm_gpu, idx_gu)
        ax = np.abs(oracle.decode(xm_gpu[:, idx_gu], dt))
        ag, au = ax @ np.abs(oracle.decode(L16["w_gate"][idx_gu], dt)), ax @ np.abs(oracle.decode(L16["w_up"][idx_gu], dt))
    assert ulp_close(hm_gpu, oracle.silu_mul(g, u, dt), frac_exact=0.97, dt=dt, abs_err=silu_mul_err(g, u, ag, au))
    # down
    idx_d = m.idx(afx.OP_DOWN).cpu().numpy()[: stats[3][0]]
    assert np.array_equal(idx_d, expected("down", hm_gpu))
    h2_ref = h1_ref + gemv(3, cfg.hidden, hm_gpu, idx_d, L16["w_down"])
    assert rel_err(m.h.cpu().numpy(), h2_ref) <= TOL
    return dict(idx=[idx, idx_o, idx_gu, idx_d], kc=bits_np(m.k_cache[layer]), vc=bits_np(m.v_cache[layer]))


@pytest.mark.parametrize("dt,heads,kvh,mlp,use", [("bf16", 4, 2, 1024, (True, True, True, True)),
                                                  ("f16", 2, 2, 1376, (True, True, True, True)),
                                                  ("bf16", 4, 4, 1024, (True, False, True, False)),
                                                  ("bf16", 2, 1, 512, (False, True, False, True))])
def test_q4_layer_step_every_stage_matches_oracle(dt, heads, kvh, mlp, use):
    """Two layers at cross-layer depth 1 (bookkeeping: the second layer's sets are compared with the
    first's), all operators 4-bit or a mix with the 16-bit fused kernels."""
    hidden, max_seq, pos, T, NL = heads * 128, 48, 37, 1, 2
    n_qkv = (heads + 2 * kvh) * 128
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK, xl_depth=1, xl_mode=1)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    layers, q4, q4dev, caches = [], [], [], []
    for l in range(NL):
        L = synth.layer_weights(61, l, hidden, heads, kvh, mlp, dt, gain_jitter=0.1)
        L["k"] = k
        kc0, vc0 = synth.kv_cache(61, l, T, max_seq, kvh, pos)
        L["k_cache"], L["v_cache"] = kc0, vc0
        layers.append(L)
        caches.append((kc0, vc0))
        rows = q4_layer_weights(61, l, hidden, heads * 128, n_qkv, mlp)
        q4.append(rows)
        q4dev.append([torch.from_numpy(r).cuda() for r in rows])
    m = make(cfg, layers, T, afx.MODE_TOPK, xl_depth=1, xl_mode=afx.XL_BOOKKEEP, max_seq=max_seq)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    h = synth.hidden_state(61, 5, T, hidden, scales_stream=6)
    m.h.copy_(torch.from_numpy(h).cuda())
    prev = None
    for l in range(NL):
        afx.afx_layer_step_q4(m.handle, l, m.state, pos, q4_struct(q4dev[l], use), dev_status=status)
        torch.cuda.synchronize()
        out = check_q4_stages(cfg, layers[l], q4[l], use, oracle_weights(layers[l], k), m, l, h, caches[l][0],
                              caches[l][1], pos)
        assert [len(i) for i in out["idx"]] == k
        if prev is not None:  # bookkeeping against the previous layer's sets
            stats = m.stats.cpu().numpy()[l]
            for op, K in enumerate(m.K_op):
                miss, hit = oracle.diff_active(out["idx"][op], prev[op], K)
                assert stats[op][1] == hit and stats[op][2] == miss.size
                assert np.array_equal(m.miss(op).cpu().numpy()[: miss.size], miss)
        prev = out["idx"]
        h = m.h.cpu().numpy().copy()
    assert int(status.item()) == 0
    m.close()


def test_q4_layer_step_reuses_the_predictor_layers_sets():
    """Four layers at depth 3, REUSE: layers 1 and 2 compute on layer 0's sets, layer 3 selects again."""
    dt, heads, kvh, mlp, T, max_seq, pos, NL = "bf16", 4, 2, 1024, 1, 32, 20, 4
    hidden, n_qkv = heads * 128, (heads + 2 * kvh) * 128
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK, xl_depth=3, xl_mode=2)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    layers, q4, q4dev, caches = [], [], [], []
    for l in range(NL):
        L = synth.layer_weights(64, l, hidden, heads, kvh, mlp, dt, gain_jitter=0.1)
        L["k"] = k
        kc0, vc0 = synth.kv_cache(64, l, T, max_seq, kvh, pos)
        L["k_cache"], L["v_cache"] = kc0, vc0
        layers.append(L)
        caches.append((kc0, vc0))
        rows = q4_layer_weights(64, l, hidden, heads * 128, n_qkv, mlp)
        q4.append(rows)
        q4dev.append([torch.from_numpy(r).cuda() for r in rows])
    m = make(cfg, layers, T, afx.MODE_TOPK, xl_depth=3, xl_mode=afx.XL_REUSE, max_seq=max_seq)
    h = synth.hidden_state(64, 5, T, hidden, scale=4.0, scales_stream=6)
    m.h.copy_(torch.from_numpy(h).cuda())
    use = (True, True, True, True)
    pred = None
    for l in range(NL):
        afx.afx_layer_step_q4(m.handle, l, m.state, pos, q4_struct(q4dev[l], use))
        torch.cuda.synchronize()
        own = l % 3 == 0
        out = check_q4_stages(cfg, layers[l], q4[l], use, oracle_weights(layers[l], k), m, l, h, caches[l][0],
                              caches[l][1], pos, lists=None if own else dict(zip(OPN, pred)))
        if own:
            pred = [i.copy() for i in out["idx"]]
        h = m.h.cpu().numpy().copy()
    m.close()


def test_q4_layer_step_at_7b_size():
    """One layer of Llama-7B shapes, all four operators 4-bit, top 50 %."""
    dt, hidden, heads, mlp, T, pos, max_seq = "bf16", 4096, 32, 11008, 1, 64, 72
    cfg = ol.Config(dt, hidden, heads, heads, mlp, mode=oracle.TOPK)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    L = synth.layer_weights(62, 0, hidden, heads, heads, mlp, dt)
    L["k"] = k
    kc0, vc0 = synth.kv_cache(62, 0, T, max_seq, heads, pos)
    L["k_cache"], L["v_cache"] = kc0, vc0
    rows = q4_layer_weights(62, 0, hidden, heads * 128, 3 * hidden, mlp)
    dev = [torch.from_numpy(r).cuda() for r in rows]
    m = make(cfg, [L], T, afx.MODE_TOPK, max_seq=max_seq)
    h = synth.hidden_state(62, 5, T, hidden, scales_stream=6)
    m.h.copy_(torch.from_numpy(h).cuda())
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    use = (True, True, True, True)
    afx.afx_layer_step_q4(m.handle, 0, m.state, pos, q4_struct(dev, use), dev_status=status)
    torch.cuda.synchronize()
    check_q4_stages(cfg, L, rows, use, oracle_weights(L, k), m, 0, h, kc0, vc0, pos)
    assert int(status.item()) == 0
    m.close()


def test_q4_layer_step_rejects_what_it_cannot_run():
    dt, heads, kvh, mlp, T = "bf16", 2, 1, 512, 2
    hidden = heads * 128
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK)
    L = synth.layer_weights(63, 0, hidden, heads, kvh, mlp, dt)
    L["k"] = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    rows = [torch.from_numpy(r).cuda() for r in q4_layer_weights(63, 0, hidden, heads * 128, (heads + 2 * kvh) * 128, mlp)]
    m = make(cfg, [L], T, afx.MODE_TOPK, max_seq=16)
    with pytest.raises(afx.AfxError) as e:  # two tokens per step
        afx.afx_layer_step_q4(m.handle, 0, m.state, 3, q4_struct(rows))
    assert e.value.status == 4
    m.close()
    m = make(cfg, [L], 1, afx.MODE_TOPK, max_seq=16)
    q = q4_struct(rows)
    q.ldq_bytes[2] = 8  # not a multiple of 16
    with pytest.raises(afx.AfxError) as e:
        afx.afx_layer_step_q4(m.handle, 0, m.state, 3, q)
    assert e.value.status == 2
    q = q4_struct(rows)
    q.ldq_bytes[3] = 16  # shorter than a row
    with pytest.raises(afx.AfxError) as e:
        afx.afx_layer_step_q4(m.handle, 0, m.state, 3, q)
    assert e.value.status == 1
    with pytest.raises(afx.AfxError):
        afx.afx_layer_step_q4(m.handle, 1, m.state, 3, q4_struct(rows))  # no such layer
    m.close()

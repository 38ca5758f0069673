"""Parity at the FULL sizes of the five workload configurations (Llama-7B / 13B / 70B shaped
layers, KV cache of 2048 positions), stage by stage against the oracle on the same stage
inputs, through the same entry points and launch shapes the benchmark times."""
import numpy as np
import pytest
import torch

import oracle
import oracle.layer as ol
from paper_2504_08378_b200 import afx, synth
from gpu_util import dev_i32, rel_err
from test_gpu_layer import OPN, TOL, bits_np, check_layer_stages, hm_close, make, oracle_weights

pytestmark = pytest.mark.gpu


def full_layer(seed, layer, hidden, heads, kvh, mlp, dt, k=None, tau=None):
    """(device dict for the model, numpy dict for the oracle) of one random-init layer."""
    dev = synth.device_layer_weights(seed, layer, hidden, heads, kvh, mlp, dt)
    host = {n: dev[n].cpu().numpy().view(np.uint16) for n in ("w_qkv", "w_o", "w_gu", "w_down")}
    host["w_gate"], host["w_up"] = synth.split_gate_up(host["w_gu"])
    host["g_attn"] = np.ones(hidden, np.float32)
    host["g_mlp"] = np.ones(hidden, np.float32)
    for d in (dev, host):
        d["k"] = k or [0, 0, 0, 0]
        d["tau"] = tau or [0.0, 0.0, 0.0, 0.0]
    return dev, host


def test_config2_mlp_block_7b_threshold_sweep():
    dt, hidden, mlp, T = "f16", 4096, 11008, 1
    cfg = ol.Config(dt, hidden, 32, 32, mlp, mode=oracle.THRESHOLD)
    dev, host = full_layer(2, 0, hidden, 32, 32, mlp, dt)
    x = synth.laplace_bits(2, 100, (T, hidden), dt)
    dense = ol.mlp_block(cfg, oracle_weights(host, None, [0, 0, -1.0, -1.0]), x)
    hm_abs = np.sort(np.abs(oracle.decode(dense["hm"], dt)).ravel())
    for p in (0, 25, 50, 70, 90):
        tau_d = -1.0 if p == 0 else float(hm_abs[(hm_abs.size * p) // 100])
        tau = [0.0, 0.0, synth.laplace_tau(p / 100.0), tau_d]
        dev["tau"] = tau
        m = make(cfg, [dev], T, afx.MODE_THRESHOLD, max_seq=8)
        xd = torch.from_numpy(x.view(np.int16)).cuda()
        y = torch.full((T, hidden), float("nan"), device="cuda")
        m.mlp_block(0, xd, y)
        torch.cuda.synchronize()
        ref = ol.mlp_block(cfg, oracle_weights(host, None, tau), x)
        stats = m.stats.cpu().numpy()[0]
        assert np.array_equal(m.idx(afx.OP_GU).cpu().numpy()[: stats[2][0]], ref["idx_gu"]), p
        if p:
            assert abs(stats[2][0] / hidden - (1 - p / 100)) < 0.03  # realised sparsity near the target
        hm_gpu = bits_np(m.bits(afx.BUF_HM))
        assert hm_close(host, dt, mlp, x, ref["idx_gu"], hm_gpu, ref["hm"]), p
        idx_d = m.idx(afx.OP_DOWN).cpu().numpy()[: stats[3][0]]
        assert np.array_equal(idx_d, oracle.select_active(hm_gpu, dt, oracle.THRESHOLD, tau=tau_d))
        y_ref = oracle.sparse_gemv(host["w_down"], dt, hidden, hm_gpu, idx_d)
        assert rel_err(y.cpu().numpy(), y_ref) <= TOL
        m.close()


def _run_layers(cfg, layers_dev, layers_host, k, T, pos, max_seq, seed, xl_depth=0, xl_mode=0, warm_tokens=0):
    kvh = cfg.n_kv_heads
    caches = []
    for l, dev in enumerate(layers_dev):
        kc0, vc0 = synth.kv_cache(seed, l, T, max_seq, kvh, pos)
        dev["k_cache"], dev["v_cache"] = kc0, vc0
        caches.append((kc0, vc0))
    m = make(cfg, layers_dev, T, afx.MODE_TOPK, xl_depth=xl_depth, xl_mode=xl_mode, max_seq=max_seq)
    for w in range(warm_tokens):  # earlier, different tokens: they leave their k-th keys as search hints
        m.h.copy_(torch.from_numpy(synth.hidden_state(seed, 105 + w, T, cfg.hidden, scales_stream=6)).cuda())
        for l in range(len(layers_host)):
            m.layer_step(l, pos)
        torch.cuda.synchronize()
        assert (m.stats.cpu().numpy()[:, :, 3] >> 16 == 1).all()
    h = synth.hidden_state(seed, 5, T, cfg.hidden, scales_stream=6)
    m.h.copy_(torch.from_numpy(h).cuda())
    prev_idx = None
    for l, host in enumerate(layers_host):
        m.layer_step(l, pos)
        torch.cuda.synchronize()
        out = check_layer_stages(cfg, host, oracle_weights(host, k), m, l, h, caches[l][0], caches[l][1], pos, T)
        if T == 1:
            assert [len(i) for i in out["idx"]] == k
        if xl_depth and l > 0:  # bookkeeping against the predictor layer's sets
            stats = m.stats.cpu().numpy()[l]
            for op, K in enumerate(m.K_op):
                miss, hit = oracle.diff_active(out["idx"][op], prev_idx[op], K)
                assert stats[op][1] == hit and stats[op][2] == miss.size
                assert np.array_equal(m.miss(op).cpu().numpy()[: miss.size], miss)
        if l == 0:
            prev_idx = out["idx"]
        h = m.h.cpu().numpy().copy()
    m.close()


def test_config3_7b_decode_layers_with_cross_layer_bookkeeping():
    dt, hidden, heads, mlp = "bf16", 4096, 32, 11008
    cfg = ol.Config(dt, hidden, heads, heads, mlp, mode=oracle.TOPK, xl_depth=3, xl_mode=1)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    pairs = [full_layer(3, l, hidden, heads, heads, mlp, dt, k=k) for l in range(2)]
    _run_layers(cfg, [p[0] for p in pairs], [p[1] for p in pairs], k, 1, 2048, 2056, 3, xl_depth=3,
                xl_mode=afx.XL_BOOKKEEP)


@pytest.mark.parametrize("dt", ["bf16", "f16"])
def test_config3_7b_layer_after_other_tokens(dt):
    """The token checked is the third one decoded: its top-k searches start from the previous
    token's k-th keys (three 8-channel chunks per thread on the 11008-wide input)."""
    hidden, heads, mlp = 4096, 32, 11008
    cfg = ol.Config(dt, hidden, heads, heads, mlp, mode=oracle.TOPK)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    dev, host = full_layer(6, 0, hidden, heads, heads, mlp, dt, k=k)
    _run_layers(cfg, [dev], [host], k, 1, 2048, 2056, 6, warm_tokens=2)


@pytest.mark.parametrize("T", [1, 4])
def test_config4_13b_layer(T):
    dt, hidden, heads, mlp = "bf16", 5120, 40, 13824
    cfg = ol.Config(dt, hidden, heads, heads, mlp, mode=oracle.TOPK)
    k = [synth.keep_count(K, 60) for K in (hidden, heads * 128, hidden, mlp)]
    dev, host = full_layer(4, 0, hidden, heads, heads, mlp, dt, k=k)
    _run_layers(cfg, [dev], [host], k, T, 2048, 2056, 4)


def test_wide_model_with_eight_tokens_per_step():
    """Hidden size 8192 with 8 tokens: the normalised inputs of 8 tokens take 128 KB of shared
    memory, so the several-token operators run with their short pipeline."""
    dt, hidden, heads, kvh, mlp = "bf16", 8192, 64, 8, 2048
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    dev, host = full_layer(7, 0, hidden, heads, kvh, mlp, dt, k=k)
    _run_layers(cfg, [dev], [host], k, 8, 40, 48, 7)


def test_config5_70b_layer_and_cached_down_projection():
    dt, hidden, heads, kvh, mlp = "bf16", 8192, 64, 8, 28672
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    dev, host = full_layer(5, 0, hidden, heads, kvh, mlp, dt, k=k)
    _run_layers(cfg, [dev], [host], k, 1, 2048, 2056, 5)
    # the down projection served from a 30 % hot-channel cache, weights in pinned host memory
    K, N = mlp, hidden
    C = (K * 30) // 100
    Wt = host["w_down"]
    pinned = torch.from_numpy(Wt.view(np.int16)).pin_memory()
    slots = torch.zeros((C + k[3], N), dtype=torch.int16, device="cuda")
    handle = afx.afx_cache_create(afx.CacheDesc(dtype=afx.DTYPES[dt], K=K, N=N, ldw=N, capacity=C, staging_rows=k[3],
                                                host_base=pinned.data_ptr(), slots=slots.data_ptr()))
    oc = oracle.LfuCache(K, C)
    slot_out = torch.empty(K, dtype=torch.int32, device="cuda")
    stats = torch.zeros(3, dtype=torch.int64, device="cuda")
    y = torch.empty((1, N), dtype=torch.float32, device="cuda")
    for s in range(4):
        x = synth.zipf_activity_bits(5, 300 + s, K, dt, alpha=1.1, perm_stream=9)
        active = oracle.select_active(x, dt, oracle.TOPK, k=k[3])
        want = oc.step(active)
        idx, cnt = dev_i32(active), dev_i32([active.size])
        afx.afx_cache_fetch(handle, idx, cnt, slot_out, stats)
        afx.afx_sparse_gemv(slots, dt, K, N, N, torch.from_numpy(x.view(np.int16)).cuda(), 1, idx, cnt, slot_out, y, 0)
        torch.cuda.synchronize()
        st = afx.CacheStats.from_buffer_copy(stats.cpu().numpy().tobytes())
        assert (st.hits, st.misses, st.transients, st.overflow) == (want["hits"], want["misses"], want["transients"], 0)
        assert np.array_equal(slot_out[: active.size].cpu().numpy(), want["slot"])
        assert rel_err(y.cpu().numpy(), oracle.sparse_gemv(Wt, dt, N, x, active)) <= TOL
    afx.afx_cache_destroy(handle)

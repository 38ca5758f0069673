"""Cross-layer prediction past the first group, and launch chains without synchronisation.

(1) Eight small layers at depth 3 and depth 1, bookkeeping and reuse: predictions published by
    layers 3 and 6 are consumed, the double-buffered predicted sets flip several times, the
    last group is clipped.  Free-running GPU against the free-running oracle.
(2) The same chain enqueued in one go, several tokens back to back, must give the bits of the
    run that synchronises after every layer step: kernels overlap their prologues with their
    predecessors' tails, and everything a prologue reads early must already be final.
(3) Reuse at Llama-7B size across a group boundary (layers 2, 3, 4), stage by stage.
"""
import numpy as np
import pytest
import torch

import oracle
import oracle.layer as ol
from paper_2504_08378_b200 import afx, synth
from gpu_util import rel_err
from test_gpu_configs import full_layer
from test_gpu_layer import OPN, TOL, bits_np, check_layer_stages, make, oracle_weights

pytestmark = pytest.mark.gpu


def small_model(seed, n_layers, dt, heads, kvh, mlp, T, max_seq, pos, depth, xl_mode, percent=50):
    hidden = heads * 128
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK, xl_depth=depth, xl_mode=xl_mode)
    k = [synth.keep_count(K, percent) for K in (hidden, heads * 128, hidden, mlp)]
    layers, lws, caches = [], [], []
    for l in range(n_layers):
        L = synth.layer_weights(seed, l, hidden, heads, kvh, mlp, dt, gain_jitter=0.1)
        L["k"] = k
        kc0, vc0 = synth.kv_cache(seed, l, T, max_seq, kvh, pos)
        L["k_cache"], L["v_cache"] = kc0, vc0
        layers.append(L)
        lws.append(oracle_weights(L, k))
        caches.append((kc0.copy(), vc0.copy()))
    m = make(cfg, layers, T, afx.MODE_TOPK, xl_depth=depth, xl_mode=xl_mode, max_seq=max_seq)
    return cfg, k, layers, lws, caches, m


@pytest.mark.parametrize("xl_mode", [afx.XL_BOOKKEEP, afx.XL_REUSE])
@pytest.mark.parametrize("depth", [3, 1])
def test_eight_layers_free_running_against_the_oracle(depth, xl_mode):
    dt, heads, kvh, mlp, T, max_seq, pos, NL = "bf16", 4, 2, 1024, 1, 32, 20, 8
    cfg, k, layers, lws, caches, m = small_model(43, NL, dt, heads, kvh, mlp, T, max_seq, pos, depth, xl_mode)
    h0 = synth.hidden_state(43, 5, T, cfg.hidden, scale=4.0, scales_stream=6)
    m.h.copy_(torch.from_numpy(h0).cuda())
    xl = ol.CrossLayer(cfg)
    h = h0.astype(np.float64)
    consumed = set()
    for l in range(NL):
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
                consumed.add(depth * ((l - 1) // depth))
                assert stats[op][1] == rec["hit_" + name] and stats[op][2] == rec["miss_" + name].size, (l, name)
                assert np.array_equal(m.miss(op).cpu().numpy()[: stats[op][2]], rec["miss_" + name]), (l, name)
        assert rel_err(m.h.cpu().numpy(), h) <= TOL, l
    if xl_mode == afx.XL_BOOKKEEP:  # predictions of later predictor layers were really used
        assert consumed == ({0, 3, 6} if depth == 3 else set(range(7)))
    m.close()


def run_tokens(m, h0, n_tokens, NL, pos, sync):
    """n_tokens decode steps at successive positions; each token starts from the residual the
    previous one left (any input will do: both runs see the same).  Returns everything a
    race could corrupt."""
    m.blob.zero_()
    for l in range(NL):
        m.k_cache[l][:, pos:] = 0
        m.v_cache[l][:, pos:] = 0
    m.h.copy_(torch.from_numpy(h0).cuda())
    torch.cuda.synchronize()
    for t in range(n_tokens):
        for l in range(NL):
            m.layer_step(l, pos + t)
            if sync:
                torch.cuda.synchronize()
    torch.cuda.synchronize()
    return dict(h=m.h.cpu().numpy().copy(), stats=m.stats.cpu().numpy().copy(),
                miss=[m.miss(op).cpu().numpy().copy() for op in range(4)],
                idx=[m.idx(op).cpu().numpy().copy() for op in range(4)],
                kc=[bits_np(c).copy() for c in m.k_cache], vc=[bits_np(c).copy() for c in m.v_cache])


@pytest.mark.parametrize("NL,depth,xl_mode,heads,mlp", [(8, 3, afx.XL_BOOKKEEP, 2, 512), (8, 1, afx.XL_BOOKKEEP, 2, 512),
                                                        (8, 3, afx.XL_REUSE, 2, 512), (1, 1, afx.XL_BOOKKEEP, 1, 256),
                                                        (2, 1, afx.XL_BOOKKEEP, 1, 256)])
def test_chain_without_synchronisation_gives_the_same_bits(NL, depth, xl_mode, heads, mlp):
    """Small shapes on purpose: many of these grids fit on the device at once, so a prologue
    that read something its writer had not finished would show up as different bits.  With
    one layer the attention kernel reads cache row pos-1 written five launches earlier, and
    at depth 1 every predicted set was published exactly one layer step earlier."""
    dt, kvh, T, max_seq, pos, n_tokens = "bf16", 1, 1, 40, 20, 6
    cfg, k, layers, lws, caches, m = small_model(47, NL, dt, heads, kvh, mlp, T, max_seq, pos, depth, xl_mode)
    h0 = synth.hidden_state(47, 5, T, cfg.hidden, scale=4.0, scales_stream=6)
    ref = run_tokens(m, h0, n_tokens, NL, pos, sync=True)
    for attempt in range(5):
        got = run_tokens(m, h0, n_tokens, NL, pos, sync=False)
        assert np.array_equal(got["h"].view(np.uint32), ref["h"].view(np.uint32)), attempt
        assert np.array_equal(got["stats"], ref["stats"]), attempt
        for op in range(4):
            n_miss, n_idx = ref["stats"][NL - 1][op][2], ref["stats"][NL - 1][op][0]
            assert np.array_equal(got["miss"][op][:n_miss], ref["miss"][op][:n_miss])
            assert np.array_equal(got["idx"][op][:n_idx], ref["idx"][op][:n_idx])
        for l in range(NL):
            assert np.array_equal(got["kc"][l], ref["kc"][l]) and np.array_equal(got["vc"][l], ref["vc"][l])
    m.close()


@pytest.mark.parametrize("T,depth", [(4, 1), (8, 0), (2, 3)])
def test_chain_without_synchronisation_with_several_tokens_per_step(T, depth):
    """The same with several tokens per step: the blocks of a cluster exchange the per-token
    sets through distributed shared memory and the streaming stage runs on the tensor cores;
    launches that overlap must still give the bits of the synchronised run."""
    dt, NL, heads, kvh, mlp, max_seq, pos, n_tokens = "bf16", 4, 2, 1, 512, 40, 20, 4
    xl_mode = afx.XL_BOOKKEEP if depth else afx.XL_OFF
    cfg, k, layers, lws, caches, m = small_model(49, NL, dt, heads, kvh, mlp, T, max_seq, pos, depth, xl_mode)
    h0 = synth.hidden_state(49, 5, T, cfg.hidden, scale=4.0, scales_stream=6)
    ref = run_tokens(m, h0, n_tokens, NL, pos, sync=True)
    for attempt in range(4):
        got = run_tokens(m, h0, n_tokens, NL, pos, sync=False)
        assert np.array_equal(got["h"].view(np.uint32), ref["h"].view(np.uint32)), attempt
        assert np.array_equal(got["stats"], ref["stats"]), attempt
        for op in range(4):
            n_idx = ref["stats"][NL - 1][op][0]
            assert np.array_equal(got["idx"][op][:n_idx], ref["idx"][op][:n_idx])
        for l in range(NL):
            assert np.array_equal(got["kc"][l], ref["kc"][l]) and np.array_equal(got["vc"][l], ref["vc"][l])
    m.close()


def test_one_layer_several_tokens_each_against_the_oracle():
    """One layer stepped over successive positions: every token's stages against the oracle on
    the cache the GPU has built so far (rows written by earlier tokens are read back)."""
    dt, heads, kvh, mlp, T, max_seq, pos = "f16", 2, 1, 512, 1, 40, 20
    cfg, k, layers, lws, caches, m = small_model(48, 1, dt, heads, kvh, mlp, T, max_seq, pos, 0, afx.XL_OFF)
    h = synth.hidden_state(48, 5, T, cfg.hidden, scales_stream=6)
    kc, vc = caches[0]
    for t in range(4):
        m.h.copy_(torch.from_numpy(h).cuda())
        m.layer_step(0, pos + t)
        torch.cuda.synchronize()
        out = check_layer_stages(cfg, layers[0], lws[0], m, 0, h, kc, vc, pos + t, T)
        kc, vc = out["kc"].copy(), out["vc"].copy()
        h = synth.hidden_state(48, 6 + t, T, cfg.hidden, scales_stream=6)
    m.close()


def test_reuse_at_7b_size_across_a_group_boundary():
    """Layers 0..4 of the 7B-shaped stack at depth 3, REUSE: layers 1 and 2 compute on layer 0's
    sets, layer 3 selects for itself (and is compared with layer 0's sets), layer 4 computes on
    layer 3's.  Every stage teacher-forced against the oracle with the list it must have used."""
    dt, hidden, heads, mlp, T, pos, max_seq = "bf16", 4096, 32, 11008, 1, 2048, 2056
    cfg = ol.Config(dt, hidden, heads, heads, mlp, mode=oracle.TOPK, xl_depth=3, xl_mode=2)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    pairs = [full_layer(3, l, hidden, heads, heads, mlp, dt, k=k) for l in range(5)]
    caches = []
    for l, (dev, host) in enumerate(pairs):
        kc0, vc0 = synth.kv_cache(3, l, T, max_seq, heads, pos)
        dev["k_cache"], dev["v_cache"] = kc0, vc0
        caches.append((kc0, vc0))
    m = make(cfg, [p[0] for p in pairs], T, afx.MODE_TOPK, xl_depth=3, xl_mode=afx.XL_REUSE, max_seq=max_seq)
    h = synth.hidden_state(3, 5, T, hidden, scales_stream=6)
    m.h.copy_(torch.from_numpy(h).cuda())
    pred = None
    for l, (dev, host) in enumerate(pairs):
        m.layer_step(l, pos)
        torch.cuda.synchronize()
        own = l % 3 == 0
        out = check_layer_stages(cfg, host, oracle_weights(host, k), m, l, h, caches[l][0], caches[l][1], pos, T,
                                 lists=None if own else dict(zip(OPN, pred)))
        if l == 3:  # a predictor layer that is itself predicted: bookkeeping against layer 0's sets
            stats = m.stats.cpu().numpy()[l]
            for op, K in enumerate(m.K_op):
                miss, hit = oracle.diff_active(out["idx"][op], pred[op], K)
                assert stats[op][1] == hit and stats[op][2] == miss.size
                assert np.array_equal(m.miss(op).cpu().numpy()[: miss.size], miss)
        if own:
            pred = [i.copy() for i in out["idx"]]
        h = m.h.cpu().numpy().copy()
    m.close()

"""afx_layer_step_hosted: a decoder layer whose operators live in host memory behind the LFU
cache or the cross-layer-group swapping object, stage by stage against the oracle (the same
checks as for the fused layer step), over several layers and tokens, with preloads requested
from the state's own active lists between layer steps."""
import numpy as np
import pytest
import torch

import oracle
import oracle.layer as ol
from paper_2504_08378_b200 import afx, synth
from test_gpu_layer import OPN, check_layer_stages, make, oracle_weights

pytestmark = pytest.mark.gpu


def pinned_bits(a):
    t = torch.from_numpy(np.ascontiguousarray(a, np.uint16).view(np.int16)).pin_memory()
    return t


@pytest.mark.parametrize("dt,T,kinds", [("bf16", 1, ("cache", "swap", "cache", "swap")),
                                        ("f16", 1, ("swap", "cache", "swap", "cache")),
                                        ("bf16", 2, ("swap", None, "cache", None))])
def test_hosted_layer_step_matches_the_oracle(dt, T, kinds):
    heads, kvh, mlp, NL, max_seq, pos, d = 4, 2, 1024, 4, 32, 20, 2
    hidden = heads * 128
    cfg = ol.Config(dt, hidden, heads, kvh, mlp, mode=oracle.TOPK, xl_depth=0, xl_mode=0)
    k = [synth.keep_count(K, 50) for K in (hidden, heads * 128, hidden, mlp)]
    layers, lws, caches = [], [], []
    for l in range(NL):
        L = synth.layer_weights(701, l, hidden, heads, kvh, mlp, dt, gain_jitter=0.1)
        L["k"] = k
        kc0, vc0 = synth.kv_cache(701, l, T, max_seq, kvh, pos)
        L["k_cache"], L["v_cache"] = kc0, vc0
        L["w_gu"] = synth.interleave_gate_up(L["w_gate"], L["w_up"])
        layers.append(L)
        lws.append(oracle_weights(L, k))
        caches.append((kc0.copy(), vc0.copy()))
    m = make(cfg, layers, T, afx.MODE_TOPK, max_seq=max_seq)
    names = ["w_qkv", "w_o", "w_gu", "w_down"]
    K_op = m.K_op
    N_op = [m.n_qkv, hidden, 2 * mlp, hidden]
    keep, handles = [], []          # keep tensors alive; (kind, handle) to destroy
    ops_per_layer = [afx.HostedOps() for _ in range(NL)]
    for op, kind in enumerate(kinds):
        K, N = K_op[op], N_op[op]
        slot = torch.full((K,), -3, dtype=torch.int32, device="cuda")
        keep.append(slot)
        if kind == "cache":
            for l in range(NL):
                host = pinned_bits(layers[l][names[op]])
                C = (K * 3) // 5
                rows = torch.full((C + k[op], N), -1, dtype=torch.int16, device="cuda")
                h = afx.afx_cache_create(afx.CacheDesc(dtype=afx.DTYPES[dt], K=K, N=N, ldw=N, capacity=C, staging_rows=k[op],
                                                       host_base=host.data_ptr(), slots=rows.data_ptr()))
                keep += [host, rows]
                handles.append(("cache", h))
                ops_per_layer[l].cache[op] = h
                ops_per_layer[l].slot[op] = slot.data_ptr()
        elif kind == "swap":
            img = torch.empty(NL * K * N, dtype=torch.int16).pin_memory()
            afx.afx_swap_pack_host([np.ascontiguousarray(layers[l][names[op]]).ctypes.data for l in range(NL)], NL, d, K, N,
                                   img.data_ptr())
            desc = afx.SwapDesc(dtype=afx.DTYPES[dt], n_layers=NL, group=d, K=K, N=N, ldw=N, rows_pred=K, rows_miss=K,
                                host_base=img.data_ptr(), dev_rows=0)
            rows = torch.full((afx.afx_swap_device_bytes(desc) // 2,), -1, dtype=torch.int16, device="cuda")
            desc.dev_rows = rows.data_ptr()
            h = afx.afx_swap_create(desc)
            keep += [img, rows]
            handles.append(("swap", h))
            for l in range(NL):
                ops_per_layer[l].swap[op] = h
                ops_per_layer[l].slot[op] = slot.data_ptr()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for token in range(2):
        h = synth.hidden_state(701, 5 + token, T, hidden, scales_stream=6)
        m.h.copy_(torch.from_numpy(h).cuda())
        for l in range(NL):
            afx.afx_layer_step_hosted(m.handle, l, m.state, pos + token, ops_per_layer[l], dev_status=status)
            # the first layer of a group predicts the next group from its own active lists
            if l % d == 0 and l // d + 1 < (NL + d - 1) // d:
                for op, kind in enumerate(kinds):
                    if kind == "swap":
                        cnt = m.stats[l, op, 0:1]
                        afx.afx_swap_preload(ops_per_layer[l].swap[op], l // d + 1, m.idx(op), cnt, 2, dev_status=status)
            torch.cuda.synchronize()
            out = check_layer_stages(cfg, layers[l], lws[l], m, l, h, caches[l][0], caches[l][1], pos + token, T)
            caches[l] = (out["kc"].copy(), out["vc"].copy())
            h = m.h.cpu().numpy().copy()
    assert int(status.item()) == 0
    for kind, h_ in handles:
        (afx.afx_cache_destroy if kind == "cache" else afx.afx_swap_destroy)(h_)
    m.close()

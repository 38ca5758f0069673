"""Cross-layer-group swapping on the GPU against the oracle: preload of a predicted list into
device rows on the loader stream, on-demand loads of what the prediction missed, and the sparse
GEMV through the resulting slot list -- for several tokens, with everything enqueued without a
host synchronisation in between (stream events order the loader against the compute stream)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_08378_b200 import afx, synth
from gpu_util import dev_bits, dev_i32, rel_err

pytestmark = pytest.mark.gpu


def make_swap(per_layer, d, dt, rows_pred, rows_miss):
    L = len(per_layer)
    K, ldw = per_layer[0].shape
    host = torch.empty(L * K * ldw, dtype=torch.int16).pin_memory()
    afx.afx_swap_pack_host([np.ascontiguousarray(a).ctypes.data for a in per_layer], L, d, K, ldw, host.data_ptr())
    assert np.array_equal(host.numpy().view(np.uint16), oracle.pack_group_layout(per_layer, d))
    desc = afx.SwapDesc(dtype=afx.DTYPES[dt], n_layers=L, group=d, K=K, N=ldw, ldw=ldw, rows_pred=rows_pred,
                        rows_miss=rows_miss, host_base=host.data_ptr(), dev_rows=0)
    rows = torch.full((afx.afx_swap_device_bytes(desc) // 2,), -1, dtype=torch.int16, device="cuda")  # NaN patterns
    desc.dev_rows = rows.data_ptr()
    return afx.afx_swap_create(desc), host, rows


@pytest.mark.parametrize("dt,L,d,K,N,rows_pred,rows_miss,lead", [
    ("bf16", 5, 2, 96, 64, 48, 48, "first"),     # short last group, prediction from the group's first layer
    ("f16", 6, 3, 200, 72, 100, 100, "last"),    # prediction from the previous group's last layer
    ("bf16", 4, 2, 96, 64, 20, 40, "first"),     # prediction longer than its rows: cut
    ("bf16", 4, 1, 64, 64, 32, 8, "last"),       # on-demand rows run out in places
])
def test_swap_pipeline_matches_the_oracle(dt, L, d, K, N, rows_pred, rows_miss, lead):
    k = K // 2
    per_layer = [synth.weight(401, l, K, N, dt) for l in range(L)]
    handle, host, rows = make_swap(per_layer, d, dt, rows_pred, rows_miss)
    n_tokens = 3
    # activations: a shared component per token so that neighbouring layers select similar sets
    xs = [[synth.f32_to_bits((synth.laplace(402, 10 * t, (1, K)) + 0.5 * synth.laplace(402, 10 * t + l + 1, (1, K)))
                             .astype(np.float32), dt) for l in range(L)] for t in range(n_tokens)]
    lists = [[oracle.select_active(xs[t][l], dt, oracle.TOPK, k=k) for l in range(L)] for t in range(n_tokens)]
    n_groups = (L + d - 1) // d
    st = torch.cuda.Stream()
    dev = dict(x=[[dev_bits(x) for x in row] for row in xs], idx=[[dev_i32(a) for a in row] for row in lists],
               cnt=dev_i32([k]))
    slot = [[torch.full((K,), -7, dtype=torch.int32, device="cuda") for _ in range(L)] for _ in range(n_tokens)]
    stats = [[torch.zeros(4, dtype=torch.int64, device="cuda") for _ in range(L)] for _ in range(n_tokens)]
    ys = [[torch.full((1, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(L)] for _ in range(n_tokens)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    predicted = {}
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        for t in range(n_tokens):
            for l in range(L):
                g = l // d
                first, last = l == g * d, l == min(g * d + d, L) - 1
                rows_ptr = afx.afx_swap_acquire(handle, l, dev["idx"][t][l], dev["cnt"], slot[t][l], stats[t][l], stream=st,
                                                dev_status=status)
                afx.afx_sparse_gemv(rows_ptr, dt, K, N, N, dev["x"][t][l], 1, dev["idx"][t][l], dev["cnt"], slot[t][l],
                                    ys[t][l], 0, stream=st)
                if g + 1 < n_groups and ((lead == "first" and first) or (lead == "last" and last)):
                    afx.afx_swap_preload(handle, g + 1, dev["idx"][t][l], dev["cnt"], 4, stream=st, dev_status=status)
                    predicted[(t, g + 1)] = lists[t][l]
    torch.cuda.synchronize()
    any_overflow = False
    for t in range(n_tokens):
        for l in range(L):
            g = l // d
            dg = min(d, L - g * d)
            # group 0 of a later token still holds nothing new: no preload was requested for it
            P = predicted.get((t, g), [])
            want = oracle.swap_acquire(P, lists[t][l], rows_pred, rows_miss)
            got = slot[t][l].cpu().numpy()[:k]
            assert np.array_equal(got, want["slot"]), (t, l)
            sv = afx.SwapStats.from_buffer_copy(stats[t][l].cpu().numpy().tobytes())
            n_pre = min(len(P), rows_pred)
            assert (sv.hits, sv.ondemand, sv.overflow, sv.preloaded) == (want["hits"], want["ondemand"].size,
                                                                        want["overflow"], n_pre), (t, l)
            assert sv.bytes_preload == n_pre * dg * N * 2 and sv.bytes_ondemand == want["ondemand"].size * N * 2
            keep = want["slot"] >= 0
            any_overflow |= not keep.all()
            y_ref = oracle.sparse_gemv(per_layer[l], dt, N, xs[t][l], lists[t][l][keep])
            out = ys[t][l].cpu().numpy()
            assert np.isfinite(out).all() and rel_err(out, y_ref) <= 2e-3, (t, l)
    assert int(status.item()) == (3 if any_overflow else 0)
    if rows_miss == 8:
        assert any_overflow
    afx.afx_swap_destroy(handle)

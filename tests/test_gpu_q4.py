"""Sparse GEMV over 4-bit block-quantised weights on the GPU against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_08378_b200 import afx, synth
from gpu_util import dev_bits, dev_i32, rel_err

pytestmark = pytest.mark.gpu


def run(rows, K, N, x, dt, idx, count=None, accumulate=0, y0=None):
    Wq = torch.from_numpy(rows).cuda()
    y = torch.full((N,), float("nan"), dtype=torch.float32, device="cuda") if y0 is None else torch.from_numpy(y0).cuda()
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    afx.afx_sparse_gemv_q4(Wq, K, N, rows.shape[1], dev_bits(x), dt, dev_i32(idx if len(idx) else [0]),
                           dev_i32([len(idx) if count is None else count]), y, accumulate, dev_status=st)
    torch.cuda.synchronize()
    return y.cpu().numpy(), int(st.item())


@pytest.mark.parametrize("dt", ["bf16", "f16"])
@pytest.mark.parametrize("K,N", [(64, 32), (512, 1376), (300, 4096), (1024, 8192), (4096, 22016), (11008, 4096)])
def test_q4_gemv_matches_the_oracle(dt, K, N):
    rows = synth.q4_weight(601, K + N, K, N)
    x = synth.laplace_bits(601, 7, (1, K), dt)
    assert rows.shape[1] == afx.afx_q4_row_bytes(N)
    for percent in (50, 0, 90):
        k = synth.keep_count(K, percent)
        idx = oracle.select_active(x, dt, oracle.TOPK, k=k)
        y, st = run(rows, K, N, x, dt, idx)
        want = oracle.sparse_gemv_q4(rows, N, x, dt, idx)[0]
        assert st == 0 and rel_err(y, want) <= 2e-3, percent
    y0 = synth.laplace(601, 9, (N,)).astype(np.float32)
    idx = oracle.select_active(x, dt, oracle.TOPK, k=K // 2)
    y, _ = run(rows, K, N, x, dt, idx, accumulate=1, y0=y0.copy())
    assert rel_err(y, y0 + oracle.sparse_gemv_q4(rows, N, x, dt, idx)[0]) <= 2e-3
    y1, _ = run(rows, K, N, x, dt, idx, accumulate=1, y0=y0.copy())
    assert np.array_equal(y.view(np.uint32), y1.view(np.uint32))  # fixed summation order


def test_q4_gemv_exact_on_integer_data_and_edge_lists():
    """Scales that are powers of two and integer x: every product and sum is an integer in fp32."""
    K, N, dt = 48, 96, "f16"
    g = synth.rng(602, 1)
    rows = np.zeros((K, synth.q4_row_bytes(N)), np.uint8)
    rows[:, : N // 2] = g.integers(0, 256, (K, N // 2), dtype=np.uint8)
    rows[:, N // 2: N // 2 + N // 16] = np.tile(np.array([1.0, 2.0, 0.5], np.float16), (K, 1)).view(np.uint8)
    x = synth.f32_to_bits(g.integers(-4, 5, (1, K)).astype(np.float32) * 2, dt)
    idx = np.arange(0, K, 3, dtype=np.int32)
    y, st = run(rows, K, N, x, dt, idx)
    assert st == 0 and np.array_equal(y.astype(np.float64), oracle.sparse_gemv_q4(rows, N, x, dt, idx)[0])
    y, st = run(rows, K, N, x, dt, [])                       # empty list
    assert st == 0 and not y.any()
    bad = np.array([0, -3, 3, K, 6], np.int32)               # entries out of range are skipped and reported
    y, st = run(rows, K, N, x, dt, bad)
    assert st == 1 and np.array_equal(y.astype(np.float64), oracle.sparse_gemv_q4(rows, N, x, dt, [0, 3, 6])[0])
    y, st = run(rows, K, N, x, dt, np.arange(K, dtype=np.int32), count=K + 9)   # count clamped
    assert st == 3 and np.array_equal(y.astype(np.float64), oracle.sparse_gemv_q4(rows, N, x, dt, np.arange(K))[0])

"""Edge cases of the GPU path against the oracle: the largest K of the shared-memory
selection and the first K beyond it (two-pass path), all-equal and all-zero activations,
empty lists, the largest fused K, and a list whose count is zero."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_08378_b200 import afx, synth
from gpu_util import dev_bits, dev_i32, rel_err

pytestmark = pytest.mark.gpu


def run_select(x, dt, mode, k=0, tau=0.0):
    x = np.atleast_2d(x)
    T, K = x.shape
    idx = torch.full((K,), -5, dtype=torch.int32, device="cuda")
    cnt = torch.full((1,), -5, dtype=torch.int32, device="cuda")
    afx.afx_select_active(dev_bits(x), dt, K, T, mode, k, tau, idx, cnt, None)
    torch.cuda.synchronize()
    return idx.cpu().numpy()[: int(cnt.item())]


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("K", [32760, 32768, 32769, 40000, 100003])
def test_select_around_the_shared_memory_limit(dt, K):
    x = synth.laplace_bits(301, K, (2, K), dt)
    for k in (1, K // 3, K - 1):
        assert np.array_equal(run_select(x, dt, afx.MODE_TOPK, k=k), oracle.select_active(x, dt, oracle.TOPK, k=k))
    assert np.array_equal(run_select(x[0], dt, afx.MODE_THRESHOLD, tau=1.1),
                          oracle.select_active(x[0], dt, oracle.THRESHOLD, tau=1.1))


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_degenerate_activations(dt):
    K = 4096
    ones = synth.f32_to_bits(np.ones(K, np.float32), dt)
    zeros = np.zeros(K, np.uint16)
    mixed = zeros.copy()
    mixed[::7] = 0x8000  # negative zero has the same magnitude as zero
    for x in (ones, zeros, mixed):
        for k in (0, 1, 100, K // 2, K):
            got = run_select(x, dt, afx.MODE_TOPK, k=k)
            assert np.array_equal(got, np.arange(k)), k  # ties go to the lowest ids
        assert np.array_equal(run_select(x, dt, afx.MODE_THRESHOLD, tau=0.0),
                              oracle.select_active(x, dt, oracle.THRESHOLD, tau=0.0))


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_nan_and_inf_rank_by_bit_pattern(dt):
    K = 1024
    x = synth.laplace_bits(302, 1, (K,), dt)
    inf = 0x7C00 if dt == "f16" else 0x7F80
    x[5], x[77], x[500] = inf, inf | 0x8000, inf | 0x0001  # +inf, -inf, a NaN pattern
    for k in (1, 2, 3, 10):
        assert np.array_equal(run_select(x, dt, afx.MODE_TOPK, k=k), oracle.select_active(x, dt, oracle.TOPK, k=k))
    got = run_select(x, dt, afx.MODE_THRESHOLD, tau=2.0)
    assert np.array_equal(got, oracle.select_active(x, dt, oracle.THRESHOLD, tau=2.0))
    assert 500 not in got and 5 in got and 77 in got  # a NaN is never above a threshold


def test_gemv_with_an_empty_list_writes_zero_or_leaves_y():
    dt, K, N = "bf16", 256, 520
    Wt = synth.weight(303, 1, K, N, dt)
    x = synth.laplace_bits(303, 2, (1, K), dt)
    idx, cnt = dev_i32(np.zeros(K)), dev_i32([0])
    y = torch.full((1, N), 3.0, dtype=torch.float32, device="cuda")
    afx.afx_sparse_gemv(dev_bits(Wt), dt, K, N, N, dev_bits(x), 1, idx, cnt, None, y, 1)
    torch.cuda.synchronize()
    assert (y == 3.0).all()
    afx.afx_sparse_gemv(dev_bits(Wt), dt, K, N, N, dev_bits(x), 1, idx, cnt, None, y, 0)
    torch.cuda.synchronize()
    assert (y == 0.0).all()


@pytest.mark.parametrize("T", [1, 2])
def test_fused_operator_at_its_largest_k(T):
    dt, K, N = "bf16", 32768, 264
    Wt = synth.weight(304, 1, K, N, dt)
    x = synth.laplace_bits(304, 2, (T, K), dt)
    k = K // 2
    y = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
    idx = torch.full((K,), -1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    afx.afx_select_gemv(dev_bits(Wt), dt, K, N, N, dev_bits(x), T, afx.MODE_TOPK, k, 0.0, y, 0, idx, cnt)
    torch.cuda.synchronize()
    want = oracle.select_active(x, dt, oracle.TOPK, k=k)
    assert int(cnt.item()) == want.size and np.array_equal(idx.cpu().numpy()[: want.size], want)
    assert rel_err(y.cpu().numpy(), oracle.sparse_gemv(Wt, dt, N, x, want)) <= 2e-3
    with pytest.raises(afx.AfxError) as e:
        afx.afx_select_gemv(dev_bits(Wt), dt, K + 8, N, N, dev_bits(x), 1, afx.MODE_TOPK, k, 0.0, y, 0, None, None)
    assert e.value.status == 3

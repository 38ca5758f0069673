"""GPU parity: afx_select_active / afx_diff_active against the oracle, bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_08378_b200 import afx, synth
from gpu_util import dev_bits, dev_i32

pytestmark = pytest.mark.gpu

KS = [1, 8, 31, 32, 33, 512, 1000, 4096, 5120, 8192, 11008, 13824, 28672]


def run_select(x_bits, dt, mode, k=0, tau=0.0, want_bitmap=False):
    x_bits = np.atleast_2d(x_bits)
    T, K = x_bits.shape
    x = dev_bits(x_bits)
    idx = torch.full((K,), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    bm = torch.zeros(((K + 31) // 32,), dtype=torch.int32, device="cuda") if want_bitmap else None
    afx.afx_select_active(x, dt, K, T, mode, k, tau, idx, cnt, bm)
    torch.cuda.synchronize()
    n = int(cnt.item())
    out = idx.cpu().numpy()
    assert (out[n:] == -7).all(), "wrote past count"
    return (out[:n], bm.cpu().numpy().view(np.uint32)) if want_bitmap else out[:n]


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("K", KS)
def test_topk_matches_oracle(dt, K):
    x = synth.laplace_bits(101, K, (K,), dt)
    for k in sorted({0, 1, K // 2, synth.keep_count(K, 70), K - 1, K}):
        got = run_select(x, dt, afx.MODE_TOPK, k=k)
        want = oracle.select_active(x, dt, oracle.TOPK, k=k)
        assert np.array_equal(got, want), (K, k)


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("K", [33, 4096, 11008])
def test_topk_with_heavy_ties(dt, K):
    v = np.round(synth.laplace(102, K, (K,)) * 2) / 2           # a handful of distinct magnitudes
    x = synth.f32_to_bits(v.astype(np.float32), dt)
    for k in (1, K // 4, K // 2, K - 3):
        got = run_select(x, dt, afx.MODE_TOPK, k=k)
        assert np.array_equal(got, oracle.select_active(x, dt, oracle.TOPK, k=k)), (K, k)
    ones = synth.f32_to_bits(np.ones(K, np.float32), dt)        # every magnitude equal
    assert np.array_equal(run_select(ones, dt, afx.MODE_TOPK, k=K // 3), np.arange(K // 3))
    zeros = np.zeros(K, np.uint16)
    assert np.array_equal(run_select(zeros, dt, afx.MODE_TOPK, k=5), np.arange(5))


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("K", KS)
def test_threshold_matches_oracle(dt, K):
    x = synth.laplace_bits(103, K, (K,), dt)
    mags = np.abs(synth.bits_to_f32(x, dt))
    for tau in (-1.0, 0.0, synth.laplace_tau(0.25), synth.laplace_tau(0.5), float(mags[K // 2]),
                synth.laplace_tau(0.9), 1e4):
        got = run_select(x, dt, afx.MODE_THRESHOLD, tau=tau)
        want = oracle.select_active(x, dt, oracle.THRESHOLD, tau=tau)
        assert np.array_equal(got, want), (K, tau)
    assert run_select(np.zeros(K, np.uint16), dt, afx.MODE_THRESHOLD, tau=0.0).size == 0


def test_special_values():
    x = np.array([0x3C00, 0x7E00, 0x7C00, 0xFC00, 0x0000, 0x8000, 0x0001], np.uint16)
    for mode, kw in ((afx.MODE_THRESHOLD, dict(tau=0.5)), (afx.MODE_THRESHOLD, dict(tau=-1.0)),
                     (afx.MODE_TOPK, dict(k=2)), (afx.MODE_TOPK, dict(k=5))):
        got = run_select(x, "f16", mode, **kw)
        assert np.array_equal(got, oracle.select_active(x, "f16", mode, **kw))


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("T", [2, 4, 8])
def test_union_over_tokens(dt, T):
    K = 5120
    x = synth.laplace_bits(104, T, (T, K), dt)
    k = synth.keep_count(K, 60)
    got, bm = run_select(x, dt, afx.MODE_TOPK, k=k, want_bitmap=True)
    want = oracle.select_active(x, dt, oracle.TOPK, k=k)
    assert np.array_equal(got, want)
    bits = np.unpackbits(bm.view(np.uint8), bitorder="little")[:K]
    assert np.array_equal(np.flatnonzero(bits), want)
    got = run_select(x, dt, afx.MODE_THRESHOLD, tau=0.9)
    assert np.array_equal(got, oracle.select_active(x, dt, oracle.THRESHOLD, tau=0.9))


def test_diff_active_matches_oracle():
    K, dt = 4096, "bf16"
    a_scale = synth.channel_scales(7, 1, K)
    x0 = synth.f32_to_bits((synth.laplace(7, 2, (K,)) * a_scale).astype(np.float32), dt)
    x1 = synth.f32_to_bits((synth.laplace(7, 3, (K,)) * a_scale).astype(np.float32), dt)
    k = K // 2
    _, bmP = run_select(x0, dt, afx.MODE_TOPK, k=k, want_bitmap=True)
    A = run_select(x1, dt, afx.MODE_TOPK, k=k)
    P = oracle.select_active(x0, dt, oracle.TOPK, k=k)
    want_miss, want_hit = oracle.diff_active(A, P, K)
    idxA, cntA = dev_i32(A), dev_i32([A.size])
    bm = torch.from_numpy(bmP.view(np.int32)).cuda()
    miss = torch.full((K,), -1, dtype=torch.int32, device="cuda")
    mc = torch.zeros(1, dtype=torch.int32, device="cuda")
    hc = torch.zeros(1, dtype=torch.int32, device="cuda")
    afx.afx_diff_active(idxA, cntA, bm, K, miss, mc, hc)
    torch.cuda.synchronize()
    assert int(mc.item()) == want_miss.size and int(hc.item()) == want_hit
    assert np.array_equal(miss.cpu().numpy()[: want_miss.size], want_miss)
    # identical activation: nothing missed; empty list: nothing at all
    afx.afx_diff_active(dev_i32(P), dev_i32([P.size]), bm, K, miss, mc, hc)
    assert int(mc.item()) == 0 and int(hc.item()) == P.size
    afx.afx_diff_active(idxA, dev_i32([0]), bm, K, miss, mc, hc)
    assert int(mc.item()) == 0 and int(hc.item()) == 0

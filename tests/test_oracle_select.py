"""Pins for the oracle's selection: hand cases, an independent numpy brute force, invariants."""
import json
import os

import numpy as np
import pytest

import oracle
from paper_2504_08378_b200 import synth


@pytest.fixture(scope="module")
def hand(golden_dir):
    with open(os.path.join(golden_dir, "hand_cases.json")) as f:
        return json.load(f)


def _bits(vals, dt):
    return synth.f32_to_bits(np.asarray(vals, np.float32), dt)


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_hand_cases(hand, dt):
    x = _bits(hand["x"], dt)
    xn = _bits(hand["x_next"], dt)
    assert oracle.select_active(x, dt, oracle.TOPK, k=4).tolist() == hand["topk4"]["idx"]
    assert oracle.select_active(x, dt, oracle.THRESHOLD, tau=1.0).tolist() == hand["threshold1"]["idx"]
    assert oracle.select_active(x, dt, oracle.THRESHOLD, tau=-1.0).tolist() == list(range(8))
    assert oracle.select_active(xn, dt, oracle.TOPK, k=4).tolist() == hand["cross_layer"]["A"]
    both = np.stack([x, xn])
    assert oracle.select_active(both, dt, oracle.TOPK, k=4).tolist() == hand["union_T2"]
    ones = _bits(np.ones(8), dt)
    assert oracle.select_active(ones, dt, oracle.TOPK, k=3).tolist() == hand["all_equal_k3"]
    zeros = _bits(np.zeros(8), dt)
    assert oracle.select_active(zeros, dt, oracle.THRESHOLD, tau=0.0).size == 0
    assert oracle.select_active(x, dt, oracle.TOPK, k=0).size == 0
    assert oracle.select_active(x, dt, oracle.TOPK, k=8).tolist() == list(range(8))


def _numpy_topk(xbits, k):
    """Independent route: stable argsort of the negated magnitude (ties keep index order)."""
    key = (xbits & 0x7FFF).astype(np.int64)
    order = np.argsort(-key, kind="stable")
    return np.sort(order[:k]).astype(np.int32)


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("K", [1, 8, 31, 32, 33, 257, 512, 4096])
def test_topk_matches_numpy_stable_sort(dt, K):
    for trial in range(6):
        x = synth.laplace_bits(11, 1000 * K + trial, (K,), dt)
        if trial % 2:  # heavy ties: quantise magnitudes to a handful of values
            v = np.round(synth.bits_to_f32(x, dt) * 2) / 2
            x = synth.f32_to_bits(v, dt)
        for k in sorted({0, 1, K // 3, K // 2, K - 1, K}):
            if 0 <= k <= K:
                got = oracle.select_active(x, dt, oracle.TOPK, k=k)
                assert np.array_equal(got, _numpy_topk(x, k)), (K, k, trial)


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_topk_invariants(dt):
    K, k = 1000, 400
    x = synth.f32_to_bits(np.round(synth.laplace(5, 2, (K,)) * 4).astype(np.float32) / 4, dt)
    idx = oracle.select_active(x, dt, oracle.TOPK, k=k)
    key = (x & 0x7FFF).astype(np.int64)
    inside = np.zeros(K, bool)
    inside[idx] = True
    assert idx.size == k and np.all(np.diff(idx) > 0)
    assert key[inside].min() >= key[~inside].max()
    kth = key[inside].min()
    tied_in, tied_out = np.flatnonzero(inside & (key == kth)), np.flatnonzero(~inside & (key == kth))
    assert tied_out.size > 0, "case must exercise a tie at the boundary"
    assert tied_in.max() < tied_out.min()


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_threshold_is_the_elementwise_predicate(dt):
    K = 3000
    x = synth.laplace_bits(9, 4, (K,), dt)
    v = np.abs(synth.bits_to_f32(x, dt))
    for tau in (0.0, 0.25, float(v[17]), 1.0, 3.5, 100.0):
        got = oracle.select_active(x, dt, oracle.THRESHOLD, tau=tau)
        assert np.array_equal(got, np.flatnonzero(v > np.float32(tau)).astype(np.int32))
    # "above" is strict: an element equal to tau is dropped
    assert 17 not in oracle.select_active(x, dt, oracle.THRESHOLD, tau=float(v[17])).tolist()


def test_threshold_drops_nan_keeps_inf_topk_ranks_nan_first():
    x = np.array([0x3C00, 0x7E00, 0x7C00, 0xFC00, 0x0000], np.uint16)  # 1, NaN, +inf, -inf, 0
    assert oracle.select_active(x, "f16", oracle.THRESHOLD, tau=0.5).tolist() == [0, 2, 3]
    assert oracle.select_active(x, "f16", oracle.TOPK, k=2).tolist() == [1, 2]
    assert oracle.select_active(x, "f16", oracle.THRESHOLD, tau=-1.0).tolist() == [0, 1, 2, 3, 4]


def test_union_over_tokens_is_set_union():
    K, T, k = 777, 5, 200
    x = synth.laplace_bits(21, 8, (T, K), "bf16")
    per = [set(oracle.select_active(x[t], "bf16", oracle.TOPK, k=k).tolist()) for t in range(T)]
    got = oracle.select_active(x, "bf16", oracle.TOPK, k=k)
    assert got.tolist() == sorted(set().union(*per))


def test_closed_form_threshold_gives_the_target_sparsity_on_laplace_input():
    # |x| ~ Exp(1) for Laplace(0,1): P(|x| > -ln(1-p)) = 1-p
    K = 200000
    x = synth.laplace_bits(1, 77, (K,), "f16")
    for p in (0.25, 0.5, 0.7, 0.9):
        cnt = oracle.select_active(x, "f16", oracle.THRESHOLD, tau=synth.laplace_tau(p)).size
        assert abs(cnt / K - (1 - p)) < 4 * np.sqrt(p * (1 - p) / K) + 2e-3


def test_diff_active_hand_case_and_identities(hand):
    cl = hand["cross_layer"]
    miss, hit = oracle.diff_active(cl["A"], cl["P"], 8)
    assert miss.tolist() == cl["miss"] and hit == cl["hit"]
    A = np.array([1, 4, 9, 30], np.int32)
    miss, hit = oracle.diff_active(A, A, 32)
    assert miss.size == 0 and hit == 4                    # same activation: precision 1
    miss, hit = oracle.diff_active(A, np.array([0, 2, 3], np.int32), 32)
    assert miss.tolist() == A.tolist() and hit == 0       # disjoint supports: precision 0
    g = np.random.default_rng(3)
    for _ in range(20):
        a = np.sort(g.choice(500, 200, replace=False)).astype(np.int32)
        p = np.sort(g.choice(500, 260, replace=False)).astype(np.int32)
        miss, hit = oracle.diff_active(a, p, 500)
        assert miss.tolist() == sorted(set(a.tolist()) - set(p.tolist()))
        assert hit == len(set(a.tolist()) & set(p.tolist()))

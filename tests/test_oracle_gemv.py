"""Pins for the oracle's sparse GEMV: hand cases, dense brute force, algebraic identities."""
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


def _f64(bits, dt):
    return synth.bits_to_f32(bits, dt).astype(np.float64)


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_hand_cases(hand, dt):
    x = synth.f32_to_bits(np.asarray(hand["x"], np.float32), dt)
    xn = synth.f32_to_bits(np.asarray(hand["x_next"], np.float32), dt)
    Wt = synth.f32_to_bits(np.asarray(hand["W_rows"], np.float32).T.copy(), dt)  # [K=8][N=2]
    y = oracle.sparse_gemv(Wt, dt, 2, x, hand["topk4"]["idx"])
    assert y[0].tolist() == hand["topk4"]["y"]
    y = oracle.sparse_gemv(Wt, dt, 2, x, hand["threshold1"]["idx"])
    assert y[0].tolist() == hand["threshold1"]["y"]
    y = oracle.sparse_gemv(Wt, dt, 2, x, list(range(8)))
    assert y[0].tolist() == hand["dense"]["y"]
    cl = hand["cross_layer"]
    assert oracle.sparse_gemv(Wt, dt, 2, xn, cl["A"])[0].tolist() == cl["y_actual_set"]
    assert oracle.sparse_gemv(Wt, dt, 2, xn, cl["P"])[0].tolist() == cl["y_predicted_set"]


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("K,N,ldw,T", [(64, 24, 24, 1), (300, 136, 160, 3), (512, 1376, 1376, 1)])
def test_zero_sparsity_is_dense_matvec(dt, K, N, ldw, T):
    Wt = synth.weight(2, 1, K, N, dt, ldw=ldw)
    x = synth.laplace_bits(2, 2, (T, K), dt)
    y = oracle.sparse_gemv(Wt, dt, N, x, np.arange(K))
    W = _f64(Wt, dt)[:, :N]                      # [K][N]
    want = _f64(x, dt) @ W                      # library matmul on the same fp64 values
    assert np.allclose(y, want, rtol=1e-12, atol=1e-12)
    # transposed-operand mistake would show here: N != K and W is not symmetric
    assert y.shape == (T, N)


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_dense_equals_sparse_when_dropped_channels_are_zero(dt):
    K, N = 400, 96
    Wt = synth.weight(3, 1, K, N, dt)
    x = synth.laplace_bits(3, 2, (K,), dt)
    idx = oracle.select_active(x, dt, oracle.TOPK, k=150)
    xz = np.zeros_like(x)
    xz[idx] = x[idx]
    dense = oracle.sparse_gemv(Wt, dt, N, xz, np.arange(K))
    sparse = oracle.sparse_gemv(Wt, dt, N, x, idx)
    assert np.allclose(dense, sparse, rtol=0, atol=1e-13)
    assert not np.allclose(sparse, oracle.sparse_gemv(Wt, dt, N, x, np.arange(K)), atol=1e-6)


def test_one_hot_columns_copy_the_selected_activations():
    K = N = 40
    dt = "f16"
    perm = np.random.default_rng(5).permutation(K)
    W = np.zeros((K, N), np.float32)
    W[np.arange(K), perm] = 1.0                  # channel j feeds output perm[j]
    Wt = synth.f32_to_bits(W, dt)
    x = synth.laplace_bits(5, 1, (K,), dt)
    idx = np.array([0, 3, 7, 20, 39], np.int32)
    y = oracle.sparse_gemv(Wt, dt, N, x, idx)[0]
    want = np.zeros(N)
    want[perm[idx]] = _f64(x, dt)[idx]
    assert np.array_equal(y, want)


def test_small_integers_are_exact_and_order_of_idx_is_respected():
    g = np.random.default_rng(6)
    K, N = 50, 16
    W = g.integers(-8, 9, (K, N)).astype(np.float32)
    xv = g.integers(-8, 9, K).astype(np.float32)
    for dt in ("f16", "bf16"):
        Wt, x = synth.f32_to_bits(W, dt), synth.f32_to_bits(xv, dt)
        idx = np.sort(g.choice(K, 20, replace=False)).astype(np.int32)
        y = oracle.sparse_gemv(Wt, dt, N, x, idx)[0]
        want = (xv[idx].astype(np.int64)[:, None] * W[idx].astype(np.int64)).sum(0)
        assert np.array_equal(y, want.astype(np.float64))


def test_linearity_over_disjoint_lists_and_tokens_are_independent():
    K, N, dt = 256, 64, "bf16"
    Wt = synth.weight(8, 1, K, N, dt)
    x = synth.laplace_bits(8, 2, (2, K), dt)
    a = np.arange(0, K, 2, dtype=np.int32)
    b = np.arange(1, K, 2, dtype=np.int32)
    ya, yb = oracle.sparse_gemv(Wt, dt, N, x, a), oracle.sparse_gemv(Wt, dt, N, x, b)
    yab = oracle.sparse_gemv(Wt, dt, N, x, np.arange(K))
    assert np.allclose(ya + yb, yab, rtol=0, atol=1e-13)
    y0 = oracle.sparse_gemv(Wt, dt, N, x[0], a)
    assert np.array_equal(y0[0], ya[0])


def test_slot_list_redirects_the_column_but_not_the_activation():
    K, N, dt = 64, 32, "f16"
    Wt = synth.weight(9, 1, K, N, dt)
    x = synth.laplace_bits(9, 2, (K,), dt)
    idx = np.array([2, 5, 11, 40], np.int32)
    cache = Wt[[40, 2, 11, 5]].copy()            # slots 0..3 hold channels 40, 2, 11, 5
    slot = np.array([1, 3, 2, 0], np.int32)
    assert np.array_equal(oracle.sparse_gemv(cache, dt, N, x, idx, slot=slot),
                          oracle.sparse_gemv(Wt, dt, N, x, idx))


def test_padding_columns_beyond_N_are_ignored():
    K, N, ldw, dt = 32, 24, 40, "f16"
    Wt = synth.weight(10, 1, K, N, dt, ldw=ldw)
    x = synth.laplace_bits(10, 2, (K,), dt)
    y = oracle.sparse_gemv(Wt, dt, N, x, np.arange(K))
    Wt2 = Wt.copy()
    Wt2[:, N:] = 0x7BFF
    assert np.array_equal(y, oracle.sparse_gemv(Wt2, dt, N, x, np.arange(K)))

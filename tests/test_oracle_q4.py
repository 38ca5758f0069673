"""Pins for the oracle's 4-bit weight decoding and GEMV (CPU only)."""
import numpy as np

import oracle
from paper_2504_08378_b200 import synth


def test_q4_decode_hand_block():
    """One channel, one block, scale 0.5: byte m = m | ((15 - m) << 4) -> output m has code m
    (value (m - 8) / 2), output 16 + m has code 15 - m (value (7 - m) / 2)."""
    row = np.zeros((1, synth.q4_row_bytes(32)), np.uint8)
    row[0, :16] = [m | ((15 - m) << 4) for m in range(16)]
    row[0, 16:18] = np.array([0.5], np.float16).view(np.uint8)
    w = oracle.q4_decode_loops(row, 32)[0]
    assert np.array_equal(w, oracle.q4_decode(row, 32)[0])
    assert w[:16].tolist() == [(m - 8) / 2 for m in range(16)]
    assert w[16:].tolist() == [(7 - m) / 2 for m in range(16)]
    # y = x * W for a single active channel
    x = synth.f32_to_bits(np.array([3.0], np.float32), "f16")
    assert np.array_equal(oracle.sparse_gemv_q4(row, 32, x, "f16", [0])[0], 3.0 * w)


def test_q4_decode_equals_a_vectorised_numpy_decode():
    K, N = 9, 96
    rows = synth.q4_weight(81, 1, K, N)
    assert rows.shape == (K, synth.q4_row_bytes(N)) and synth.q4_row_bytes(N) == 64
    codes = rows[:, : N // 2].reshape(K, N // 32, 16)
    q = np.concatenate([codes & 0x0F, codes >> 4], axis=2).astype(np.float64)          # [K][blocks][32]
    d = rows[:, N // 2: N // 2 + N // 16].copy().view(np.float16).astype(np.float64)   # [K][blocks]
    want = ((q - 8.0) * d[:, :, None]).reshape(K, N)
    assert np.array_equal(oracle.q4_decode_loops(rows, N), want)
    assert np.array_equal(oracle.q4_decode(rows, N), want)
    assert 0 < np.abs(want).max() < 0.1 and np.unique(codes & 0x0F).size == 16


def test_q4_gemv_equals_dense_matmul_of_the_decoded_weights():
    K, N, dt = 40, 64, "bf16"
    rows = synth.q4_weight(82, 1, K, N)
    x = synth.laplace_bits(82, 2, (1, K), dt)
    W = oracle.q4_decode(rows, N)
    xv = oracle.decode(x, dt).reshape(-1)
    full = np.arange(K)
    assert np.allclose(oracle.sparse_gemv_q4(rows, N, x, dt, full)[0], xv @ W, rtol=1e-13, atol=1e-15)
    idx = np.array([1, 5, 6, 30])
    assert np.allclose(oracle.sparse_gemv_q4(rows, N, x, dt, idx)[0], xv[idx] @ W[idx], rtol=1e-13, atol=1e-15)
    assert not oracle.sparse_gemv_q4(rows, N, x, dt, []).any()
    # linearity over disjoint lists
    a, b = oracle.sparse_gemv_q4(rows, N, x, dt, [1, 5]), oracle.sparse_gemv_q4(rows, N, x, dt, [6, 30])
    assert np.allclose(a + b, oracle.sparse_gemv_q4(rows, N, x, dt, idx), rtol=1e-13, atol=1e-15)

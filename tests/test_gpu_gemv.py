"""GPU parity: afx_sparse_gemv against the fp64 oracle (max relative error 2e-3)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_08378_b200 import afx, synth
from gpu_util import dev_bits, dev_i32, rel_err

pytestmark = pytest.mark.gpu

TOL = 2e-3  # max_i |y_i - ref_i| / max(|ref_i|, rms(ref)), fp32 sums vs fp64


def run_gemv(Wt_bits, dt, N, x_bits, idx, slot=None, y0=None):
    x_bits = np.atleast_2d(x_bits)
    T, K = x_bits.shape
    ldw = Wt_bits.shape[1]
    W, x = dev_bits(Wt_bits), dev_bits(x_bits)
    cap = max(K, 1)
    idx_d = torch.zeros((cap,), dtype=torch.int32, device="cuda")
    idx_d[: len(idx)] = dev_i32(idx)
    cnt = dev_i32([len(idx)])
    slot_d = None
    if slot is not None:
        slot_d = torch.zeros((cap,), dtype=torch.int32, device="cuda")
        slot_d[: len(slot)] = dev_i32(slot)
    if y0 is None:
        y = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
        acc = 0
    else:
        y = torch.from_numpy(np.ascontiguousarray(y0, np.float32)).cuda()
        acc = 1
    afx.afx_sparse_gemv(W, dt, K, N, ldw, x, T, idx_d, cnt, slot_d, y, acc)
    torch.cuda.synchronize()
    return y.cpu().numpy()


SHAPES = [  # K, N, ldw
    (8, 8, 8), (31, 24, 24), (64, 264, 272), (512, 1376, 1376), (1000, 4096, 4096),
    (4096, 2048 + 40, 2048 + 40), (2048, 11008, 11008),
]


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("K,N,ldw", SHAPES)
def test_gemv_matches_oracle_at_several_sparsities(dt, K, N, ldw):
    Wt = synth.weight(201, K * 7 + N, K, N, dt, ldw=ldw)
    x = synth.laplace_bits(202, K, (K,), dt)
    for k in sorted({0, 1, synth.keep_count(K, 50), synth.keep_count(K, 90), K}):
        idx = oracle.select_active(x, dt, oracle.TOPK, k=k)
        y = run_gemv(Wt, dt, N, x, idx)
        ref = oracle.sparse_gemv(Wt, dt, N, x, idx)
        assert y.shape == ref.shape and np.isfinite(y).all()
        assert rel_err(y, ref) <= TOL, (K, N, k, rel_err(y, ref))
        if k == 0:
            assert (y == 0).all()


def test_config1_single_projection():
    """W fp16 512x1376, x Laplace(0,1), keep the top 50% of channels."""
    dt, K, N = "f16", 512, 1376
    Wt = synth.weight(1, 1, K, N, dt)
    x = synth.laplace_bits(1, 2, (K,), dt)
    x_d = dev_bits(x)
    idx_d = torch.zeros(K, dtype=torch.int32, device="cuda")
    cnt_d = torch.zeros(1, dtype=torch.int32, device="cuda")
    afx.afx_select_active(x_d, dt, K, 1, afx.MODE_TOPK, 256, 0.0, idx_d, cnt_d)
    idx = oracle.select_active(x, dt, oracle.TOPK, k=256)
    assert int(cnt_d.item()) == 256 and np.array_equal(idx_d.cpu().numpy()[:256], idx)
    y = torch.empty((1, N), dtype=torch.float32, device="cuda")
    afx.afx_sparse_gemv(dev_bits(Wt), dt, K, N, N, x_d, 1, idx_d, cnt_d, None, y, 0)
    torch.cuda.synchronize()
    assert rel_err(y.cpu().numpy(), oracle.sparse_gemv(Wt, dt, N, x, idx)) <= TOL


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("T", [2, 3, 4, 8])
def test_multi_token_union(dt, T):
    K, N = 1536, 2304 + 8
    Wt = synth.weight(203, T, K, N, dt)
    x = synth.laplace_bits(204, T, (T, K), dt)
    idx = oracle.select_active(x, dt, oracle.TOPK, k=synth.keep_count(K, 60))
    y = run_gemv(Wt, dt, N, x, idx)
    ref = oracle.sparse_gemv(Wt, dt, N, x, idx)
    assert rel_err(y, ref) <= TOL


def test_accumulate_adds_to_y_and_results_are_reproducible():
    dt, K, N = "bf16", 2048, 4096
    Wt = synth.weight(205, 1, K, N, dt)
    x = synth.laplace_bits(205, 2, (K,), dt)
    idx = oracle.select_active(x, dt, oracle.THRESHOLD, tau=synth.laplace_tau(0.5))
    ref = oracle.sparse_gemv(Wt, dt, N, x, idx)
    y0 = synth.laplace(205, 3, (1, N)).astype(np.float32)
    for _ in range(3):
        y = run_gemv(Wt, dt, N, x, idx, y0=y0)
        assert rel_err(y, ref + y0) <= TOL
    y_a = run_gemv(Wt, dt, N, x, idx)
    y_b = run_gemv(Wt, dt, N, x, idx)
    assert np.array_equal(y_a, y_b), "sums must not depend on block timing"


def test_slot_list_reads_columns_from_a_cache():
    dt, K, N = "f16", 600, 520
    Wt = synth.weight(206, 1, K, N, dt)
    x = synth.laplace_bits(206, 2, (K,), dt)
    idx = oracle.select_active(x, dt, oracle.TOPK, k=200)
    perm = np.random.default_rng(1).permutation(idx.size).astype(np.int32)
    cache = np.zeros((idx.size, N), np.uint16)
    cache[perm] = Wt[idx]                              # column idx[c] lives in slot perm[c]
    y = run_gemv(cache, dt, N, x, idx, slot=perm)
    assert rel_err(y, oracle.sparse_gemv(Wt, dt, N, x, idx)) <= TOL


def test_dense_equals_sparse_when_dropped_channels_are_zero():
    dt, K, N = "bf16", 1024, 1024
    Wt = synth.weight(207, 1, K, N, dt)
    x = synth.laplace_bits(207, 2, (K,), dt)
    idx = oracle.select_active(x, dt, oracle.TOPK, k=300)
    xz = np.zeros_like(x)
    xz[idx] = x[idx]
    dense = run_gemv(Wt, dt, N, xz, np.arange(K))
    sparse = run_gemv(Wt, dt, N, x, idx)
    assert rel_err(dense, sparse.astype(np.float64)) <= 1e-5


def test_integer_weights_give_exact_results():
    g = np.random.default_rng(6)
    K, N = 300, 264
    W = g.integers(-8, 9, (K, N)).astype(np.float32)
    xv = g.integers(-8, 9, K).astype(np.float32)
    for dt in ("f16", "bf16"):
        idx = np.sort(g.choice(K, 120, replace=False)).astype(np.int32)
        y = run_gemv(synth.f32_to_bits(W, dt), dt, N, synth.f32_to_bits(xv, dt), idx)
        assert np.array_equal(y[0].astype(np.float64),
                              oracle.sparse_gemv(synth.f32_to_bits(W, dt), dt, N,
                                                 synth.f32_to_bits(xv, dt), idx)[0])


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("K,N,T", [(512, 1376, 1), (4096, 2048 + 40, 1), (1000, 4096, 3), (2048, 11008, 1)])
def test_select_gemv_equals_select_then_gemv(dt, K, N, T):
    """The one-kernel form: list bit-exact, y within tolerance of the oracle."""
    Wt = synth.weight(211, K + N, K, N, dt)
    x = synth.laplace_bits(212, K, (T, K), dt)
    W, xd = dev_bits(Wt), dev_bits(x)
    for mode, kw in ((afx.MODE_TOPK, dict(k=synth.keep_count(K, 50))), (afx.MODE_TOPK, dict(k=0)),
                     (afx.MODE_THRESHOLD, dict(tau=synth.laplace_tau(0.7))), (afx.MODE_THRESHOLD, dict(tau=-1.0))):
        idx_d = torch.full((K,), -3, dtype=torch.int32, device="cuda")
        cnt_d = torch.full((1,), -3, dtype=torch.int32, device="cuda")
        y = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
        afx.afx_select_gemv(W, dt, K, N, N, xd, T, mode, kw.get("k", 0), kw.get("tau", 0.0), y, 0, idx_d, cnt_d)
        torch.cuda.synchronize()
        want = oracle.select_active(x, dt, mode, **kw)
        n = int(cnt_d.item())
        assert n == want.size and np.array_equal(idx_d.cpu().numpy()[:n], want)
        assert rel_err(y.cpu().numpy(), oracle.sparse_gemv(Wt, dt, N, x, want)) <= TOL


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_select_gemv_hint_slot(dt):
    """kth_hint: the call records 0x10000 | k-th key; whatever it finds there first (nothing, the
    exact key, a near or far key, garbage) the list and y are the same."""
    K, N, T = 4096, 1024 + 24, 1
    k = synth.keep_count(K, 50)
    Wt = synth.weight(221, 1, K, N, dt)
    x = synth.laplace_bits(222, 2, (T, K), dt)
    W, xd = dev_bits(Wt), dev_bits(x)
    want = oracle.select_active(x, dt, afx.MODE_TOPK, k=k)
    y_ref = oracle.sparse_gemv(Wt, dt, N, x, want)
    keys = np.sort(x.reshape(-1).astype(np.int64) & 0x7FFF)
    exact = int(keys[K - k])
    slot = torch.zeros(1, dtype=torch.int32, device="cuda")
    for preset in (0, None, 0x10000 | (exact + 3), 0x10000 | max(0, exact - 2000), 0x10000 | 0x7FFF, 0x7FFF, -1):
        if preset is not None:  # None: keep what the previous call recorded (the exact key)
            slot.fill_(preset)
        idx_d = torch.full((K,), -3, dtype=torch.int32, device="cuda")
        cnt_d = torch.full((1,), -3, dtype=torch.int32, device="cuda")
        y = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
        afx.afx_select_gemv(W, dt, K, N, N, xd, T, afx.MODE_TOPK, k, 0.0, y, 0, idx_d, cnt_d, kth_hint=slot)
        torch.cuda.synchronize()
        assert int(slot.item()) == 0x10000 | exact, preset
        assert int(cnt_d.item()) == k and np.array_equal(idx_d.cpu().numpy()[:k], want), preset
        assert rel_err(y.cpu().numpy(), y_ref) <= TOL, preset


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("T,K,N,n_active", [
    (2, 40, 8, 0), (2, 40, 8, 1), (3, 300, 264, 31), (5, 300, 264, 33),      # one narrow tile + a ragged one; lists around one 32-channel stage
    (4, 5000, 520, 2049), (8, 5000, 520, 4100),                              # more entries than one staged pass holds (2 and 3 passes)
    (7, 777, 1376, 777), (2, 2048, 2304 + 8, 1000),                          # every channel active; several tiles and a tail
])
def test_several_tokens_on_the_tensor_cores_edges(dt, T, K, N, n_active):
    """afx_sparse_gemv with 2..8 tokens multiplies on the tensor cores: lists that end inside a
    16-channel step, empty lists, passes beyond the staged capacity, ragged last tiles, token
    counts that leave rows of the 8-token operand empty."""
    Wt = synth.weight(210, T, K, N, dt)
    x = synth.laplace_bits(211, T, (T, K), dt)
    idx = np.sort(np.random.default_rng(K + n_active).choice(K, n_active, replace=False)).astype(np.int32)
    y = run_gemv(Wt, dt, N, x, idx)
    ref = oracle.sparse_gemv(Wt, dt, N, x, idx)
    if n_active == 0:
        assert not y.any()
    else:
        assert rel_err(y, ref) <= TOL
    y0 = synth.laplace(212, T, (T, N)).astype(np.float32)
    assert rel_err(run_gemv(Wt, dt, N, x, idx, y0=y0), ref + y0) <= TOL
    assert np.array_equal(run_gemv(Wt, dt, N, x, idx), y), "the same inputs give the same bits"


def test_several_tokens_slot_list_bad_entries_and_nan_inputs():
    """The several-token kernel keeps the list kernel's rules: slot indirection, skipped entries
    reported through the status word, and a NaN input of a channel that is NOT in the list, or a
    NaN weight row nobody asked for, never reaches y (rows behind the list's end are zero-filled
    in shared memory and meet zero inputs)."""
    dt, T, K, N = "bf16", 4, 200, 264
    Wt = synth.weight(213, 1, K, N, dt)
    x = synth.laplace_bits(213, 2, (T, K), dt)
    good = np.array([3, 10, 11, 50, 95, 96, 130, 199], np.int32)
    x[:, 7] = 0x7FC0  # NaN inputs at channels outside the list
    x[:, 150] = 0xFF80  # -inf
    guard = 4
    buf = torch.full((K + 2 * guard, N), -1, dtype=torch.int16, device="cuda")  # 0xFFFF = a NaN pattern
    buf[guard:guard + K] = dev_bits(Wt)
    W = buf[guard:guard + K]
    y = torch.empty((T, N), dtype=torch.float32, device="cuda")

    def gemv(idx, count, slot=None, rows=W):
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        afx.afx_sparse_gemv(rows, dt, K, N, N, dev_bits(x), T, dev_i32(idx), dev_i32([count]),
                            None if slot is None else dev_i32(slot), y, 0, dev_status=st)
        torch.cuda.synchronize()
        return int(st.item()), y.cpu().numpy()

    ref = oracle.sparse_gemv(Wt, dt, N, x, good)
    st, out = gemv(good, good.size)
    assert st == 0 and np.isfinite(out).all() and rel_err(out, ref) <= TOL
    st, out = gemv(np.array([3, -1, 10, 11, 50, 200, 95, 96, 1 << 30, 130, 199], np.int32), 11)
    assert st == 1 and np.isfinite(out).all() and rel_err(out, ref) <= TOL
    # slots: the listed channels' rows sit permuted in a small cache; two of them found no row
    perm = np.array([5, 2, 7, 0, 1, 6, 3, 4], np.int32)
    cache = np.full((8, N), 0xFFFF, np.uint16)
    cache[perm] = Wt[good]
    slot = perm.copy()
    slot[[1, 6]] = -1
    keep = np.array([0, 2, 3, 4, 5, 7])
    st, out = gemv(good, good.size, slot, rows=dev_bits(cache))
    assert st == 3 and np.isfinite(out).all()
    assert rel_err(out, oracle.sparse_gemv(Wt, dt, N, x, good[keep])) <= TOL
    full = np.arange(K, dtype=np.int32)
    full = full[(full != 7) & (full != 150)]
    padded = np.concatenate([full, np.full(K - full.size, 3, np.int32)])  # K entries: the count is clamped to K
    st, out = gemv(padded, K + 9)
    assert st == 3 and np.isfinite(out).all()

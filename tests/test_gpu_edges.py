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


@pytest.mark.parametrize("dt", ["f16", "bf16"])
@pytest.mark.parametrize("fill", ["ones", "zeros"])
def test_every_key_equal_at_the_largest_shared_memory_k(dt, fill):
    """K = 32768 equal magnitudes: one 16-bit counter of the packed key histogram has to hold
    32768 and the packed per-lane sums carry it; k at 1, K/2 and K-1, stand-alone and fused."""
    K, N = 32768, 64
    x = synth.f32_to_bits(np.ones(K, np.float32), dt) if fill == "ones" else np.zeros(K, np.uint16)
    x[1::2] |= 0x8000  # signs do not matter
    Wt = synth.weight(305, 1, K, N, dt)
    for k in (1, K // 2, K - 1):
        assert np.array_equal(run_select(x, dt, afx.MODE_TOPK, k=k), np.arange(k)), k
        y = torch.full((1, N), float("nan"), dtype=torch.float32, device="cuda")
        idx = torch.full((K,), -1, dtype=torch.int32, device="cuda")
        cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
        hint = torch.zeros(1, dtype=torch.int32, device="cuda")
        for _ in range(2):  # the second call starts from the first one's hint (window path)
            afx.afx_select_gemv(dev_bits(Wt), dt, K, N, N, dev_bits(x), 1, afx.MODE_TOPK, k, 0.0, y, 0, idx, cnt,
                                kth_hint=hint)
            torch.cuda.synchronize()
            assert int(cnt.item()) == k and np.array_equal(idx.cpu().numpy()[:k], np.arange(k))
            assert rel_err(y.cpu().numpy(), oracle.sparse_gemv(Wt, dt, N, x, np.arange(k, dtype=np.int32))) <= 2e-3
        assert int(hint.item()) == 0x10000 | (int(x[0]) & 0x7FFF)


def test_bad_list_entries_are_skipped_and_reported():
    """Lists come from caller memory: a count beyond K is clamped, a channel id outside [0, K)
    and a negative slot take no part, and the device status word says which happened.  The
    weights sit between NaN guard rows: a read outside them would poison y."""
    dt, K, N = "bf16", 96, 64
    Wt = synth.weight(306, 1, K, N, dt)
    x = synth.laplace_bits(306, 2, (1, K), dt)
    guard = 4
    buf = torch.full((K + 2 * guard, N), -1, dtype=torch.int16, device="cuda")  # 0xFFFF = a NaN pattern
    buf[guard:guard + K] = dev_bits(Wt)
    W = buf[guard:guard + K]
    good = np.array([3, 10, 11, 50, 95], np.int32)
    y = torch.empty((1, N), dtype=torch.float32, device="cuda")

    def gemv(idx, count, slot=None):
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        afx.afx_sparse_gemv(W, dt, K, N, N, dev_bits(x), 1, dev_i32(idx), dev_i32([count]),
                            None if slot is None else dev_i32(slot), y, 0, dev_status=st)
        torch.cuda.synchronize()
        return int(st.item()), y.cpu().numpy()

    st, out = gemv(good, good.size)
    assert st == 0 and rel_err(out, oracle.sparse_gemv(Wt, dt, N, x, good)) <= 2e-3
    # channel ids outside [0, K): skipped
    st, out = gemv(np.array([3, -1, 10, 11, 96, 50, 1 << 30, 95], np.int32), 8)
    assert st == 1 and rel_err(out, oracle.sparse_gemv(Wt, dt, N, x, good)) <= 2e-3
    # a count beyond K: clamped to K (the list buffer has K entries)
    full = np.arange(K, dtype=np.int32)
    st, out = gemv(full, K + 5)
    assert st == 3 and rel_err(out, oracle.sparse_gemv(Wt, dt, N, x, full)) <= 2e-3
    st, out = gemv(full, -2)
    assert st == 3 and not out.any()
    # negative slots (what afx_cache_fetch writes for a channel it could not place): skipped
    slot = np.array([0, -1, 2, -1, 4], np.int32)
    st, out = gemv(good, good.size, slot)
    keep = np.array([0, 2, 4])
    want = oracle.sparse_gemv(Wt, dt, N, x, good[keep], slot=slot[keep])
    assert st == 3 and np.isfinite(out).all() and rel_err(out, want) <= 2e-3

    # the set difference and the cache policy apply the same rule
    bitmap = np.zeros((K + 31) // 32, np.uint32)
    for j in (10, 50):
        bitmap[j >> 5] |= np.uint32(1 << (j & 31))
    lst = np.array([3, -7, 10, 11, 50, 95, 4096], np.int32)
    miss = torch.full((K,), -9, dtype=torch.int32, device="cuda")
    nm, nh, st = (torch.zeros(1, dtype=torch.int32, device="cuda") for _ in range(3))
    afx.afx_diff_active(dev_i32(lst), dev_i32([lst.size]), torch.from_numpy(bitmap.view(np.int32)).cuda(), K, miss, nm, nh,
                        dev_status=st)
    torch.cuda.synchronize()
    assert (int(nm.item()), int(nh.item()), int(st.item())) == (3, 2, 1)
    assert miss.cpu().numpy()[:3].tolist() == [3, 11, 95]


def test_gemv_after_a_cache_fetch_that_ran_out_of_staging_rows():
    """Two cache rows, one staging row, five active channels from a cold cache: two are
    installed, one is staged, two get slot -1.  The fetch reports it, and the GEMV that follows
    in the same stream leaves those two channels out instead of reading row -1."""
    dt, K, N, C, staging = "f16", 32, 64, 2, 1
    Wt = synth.weight(307, 1, K, N, dt)
    x = synth.laplace_bits(307, 2, (1, K), dt)
    pinned = torch.from_numpy(Wt.view(np.int16)).pin_memory()
    guard = 2
    buf = torch.full((C + staging + 2 * guard, N), -1, dtype=torch.int16, device="cuda")
    slots = buf[guard:guard + C + staging]
    handle = afx.afx_cache_create(afx.CacheDesc(dtype=afx.DTYPES[dt], K=K, N=N, ldw=N, capacity=C, staging_rows=staging,
                                                host_base=pinned.data_ptr(), slots=slots.data_ptr()))
    active = np.array([1, 5, 9, 20, 31], np.int32)
    slot_out = torch.full((K,), -5, dtype=torch.int32, device="cuda")
    stats = torch.zeros(3, dtype=torch.int64, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty((1, N), dtype=torch.float32, device="cuda")
    idx, cnt = dev_i32(active), dev_i32([active.size])
    afx.afx_cache_fetch(handle, idx, cnt, slot_out, stats, dev_status=st)
    afx.afx_sparse_gemv(slots, dt, K, N, N, dev_bits(x), 1, idx, cnt, slot_out, y, 0, dev_status=st)
    torch.cuda.synchronize()
    sv = afx.CacheStats.from_buffer_copy(stats.cpu().numpy().tobytes())
    assert (sv.hits, sv.misses, sv.transients, sv.overflow) == (0, 5, 3, 2)
    assert slot_out.cpu().numpy()[:5].tolist() == [0, 1, 2, -1, -1]
    assert int(st.item()) == 3
    out = y.cpu().numpy()
    assert np.isfinite(out).all()
    assert rel_err(out, oracle.sparse_gemv(Wt, dt, N, x, active[:3])) <= 2e-3
    assert (buf[:guard] == -1).all() and (buf[guard + C + staging:] == -1).all()
    afx.afx_cache_destroy(handle)

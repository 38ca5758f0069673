"""GPU parity of the hot-weight cache (afx_cache_*) with the oracle's LFU cache: slot lists,
hit/miss/transient counts, tables and fetched columns bit for bit, over many steps."""
import ctypes
import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2504_08378_b200 import afx, synth
from gpu_util import dev_i32, rel_err

pytestmark = pytest.mark.gpu


class DeviceCache:
    """Pinned host weights + device slots + the library's cache object."""

    def __init__(self, Wt_bits, dtype, capacity, staging_rows):
        K, ldw = Wt_bits.shape
        self.K, self.N, self.C = K, ldw, capacity
        self.host = torch.from_numpy(Wt_bits.view(np.int16).copy()).pin_memory()
        self.slots = torch.zeros((capacity + staging_rows, ldw), dtype=torch.int16, device="cuda")
        d = afx.CacheDesc(dtype=afx.DTYPES[dtype], K=K, N=ldw, ldw=ldw, capacity=capacity,
                          staging_rows=staging_rows, host_base=self.host.data_ptr(), slots=self.slots.data_ptr())
        self.handle = afx.afx_cache_create(d)
        self.slot_out = torch.full((K,), -7, dtype=torch.int32, device="cuda")
        self.stats = torch.zeros(3, dtype=torch.int64, device="cuda")  # 24 bytes = afx_cache_stats

    def step(self, active):
        idx = dev_i32(active)
        cnt = dev_i32([len(active)])
        afx.afx_cache_fetch(self.handle, idx, cnt, self.slot_out, self.stats)
        torch.cuda.synchronize()
        raw = self.stats.cpu().numpy().tobytes()
        st = afx.CacheStats.from_buffer_copy(raw)
        return self.slot_out[: len(active)].cpu().numpy(), st

    def close(self):
        afx.afx_cache_destroy(self.handle)


def test_paper_cache_example_on_the_gpu(golden_dir):
    with open(os.path.join(golden_dir, "cache_example.json")) as f:
        ex = json.load(f)
    K, C, N = ex["K"], ex["capacity"], 64
    Wt = synth.weight(3, 1, K, N, "f16")
    dc = DeviceCache(Wt, "f16", C, K)
    afx.afx_cache_reset(dc.handle)
    afx.afx_cache_install(dc.handle, ex["initial"])
    for tok in ex["tokens"]:
        slots, st = dc.step(tok["active"])
        assert (st.hits, st.misses, st.transients, st.overflow) == (tok["hits"], tok["misses"], 0, 0)
        assert st.bytes_fetched == tok["misses"] * N * 2
        slot_of, _ = afx.afx_cache_snapshot(dc.handle, K)
        assert np.flatnonzero(slot_of >= 0).tolist() == tok["cached_after"]
        got = dc.slots.cpu().numpy().view(np.uint16)
        for j, s in zip(tok["active"], slots):
            assert np.array_equal(got[s], Wt[j])
    dc.close()


@pytest.mark.parametrize("K,N,frac,keep,steps", [(256, 64, 0.3, 0.5, 48), (2048, 136, 0.3, 0.5, 40),
                                                 (1000, 64, 0.6, 0.25, 40), (512, 64, 1.0, 0.5, 12)])
def test_cache_steps_match_oracle_bit_for_bit(K, N, frac, keep, steps):
    dt = "bf16"
    C = max(1, int(K * frac))
    k = int(K * keep)
    Wt = synth.weight(11, K, K, N, dt)
    dc = DeviceCache(Wt, dt, C, K)
    oc = oracle.LfuCache(K, C)
    for s in range(steps):
        if s == steps // 2:  # a new sequence: usage counts restart, contents stay
            afx.afx_cache_reset(dc.handle)
            oc.reset_counts()
        x = synth.zipf_activity_bits(11, 100 + s, K, dt, alpha=1.1, perm_stream=5)
        active = oracle.select_active(x, dt, oracle.TOPK, k=k)
        want = oc.step(active)
        slots, st = dc.step(active)
        assert (st.hits, st.misses, st.transients, st.overflow) == (want["hits"], want["misses"], want["transients"], 0)
        assert np.array_equal(slots, want["slot"]), f"step {s}"
        slot_of, usage = afx.afx_cache_snapshot(dc.handle, K)
        assert np.array_equal(slot_of, oc.slot_of) and np.array_equal(usage, oc.freq)
        assert st.bytes_fetched == want["misses"] * N * 2
        # every active channel's row holds that channel's column
        rows = dc.slots.cpu().numpy().view(np.uint16)[slots]
        assert np.array_equal(rows, Wt[active])
    dc.close()


def test_gemv_through_cache_slots_matches_oracle():
    dt, K, N, C = "bf16", 2048, 264, 600
    Wt = synth.weight(13, 1, K, N, dt, ldw=272)
    dc = DeviceCache(Wt, dt, C, K)
    oc = oracle.LfuCache(K, C)
    y = torch.empty((1, N), dtype=torch.float32, device="cuda")
    for s in range(6):
        x = synth.zipf_activity_bits(13, 50 + s, K, dt)
        active = oracle.select_active(x, dt, oracle.TOPK, k=K // 2)
        oc.step(active)
        idx, cnt = dev_i32(active), dev_i32([active.size])
        xd = torch.from_numpy(x.view(np.int16)).cuda()
        afx.afx_cache_fetch(dc.handle, idx, cnt, dc.slot_out, dc.stats)
        afx.afx_sparse_gemv(dc.slots, dt, K, N, 272, xd, 1, idx, cnt, dc.slot_out, y, 0)
        torch.cuda.synchronize()
        y_ref = oracle.sparse_gemv(Wt, dt, N, x, active)
        assert rel_err(y.cpu().numpy(), y_ref) <= 2e-3
    dc.close()


def test_transients_beyond_the_staging_rows_are_reported():
    dt, K, N, C = "f16", 64, 64, 8
    Wt = synth.weight(17, 1, K, N, dt)
    dc = DeviceCache(Wt, dt, C, 4)
    slots, st = dc.step(np.arange(32))  # 8 fill the cache, 24 transients, 4 staging rows
    assert (st.hits, st.misses, st.transients, st.overflow) == (0, 32, 24, 20)
    assert (slots[:12] >= 0).all() and (slots[12:] == -1).all()
    dc.close()


def test_cache_create_rejects_bad_descriptors():
    host = torch.zeros((8, 64), dtype=torch.int16).pin_memory()
    slots = torch.zeros((8, 64), dtype=torch.int16, device="cuda")
    ok = dict(dtype=0, K=8, N=64, ldw=64, capacity=4, staging_rows=4, host_base=host.data_ptr(), slots=slots.data_ptr())

    def status(**kw):
        with pytest.raises(afx.AfxError) as e:
            afx.afx_cache_create(afx.CacheDesc(**{**ok, **kw}))
        return e.value.status

    assert status(capacity=0) == 3 and status(capacity=9) == 3
    assert status(N=60) == 2 and status(dtype=5) == 4 and status(K=0) == 1
    unpinned = np.zeros((8, 64), np.int16)
    assert status(host_base=unpinned.ctypes.data) == 1

"""Host side of the cross-layer-group swapping, without a GPU: the library's layout indexer
and packer against the oracle's (which is pinned to the paper's example)."""
import ctypes

import numpy as np
import pytest

import oracle
from paper_2504_08378_b200 import afx, synth


@pytest.mark.parametrize("L,d,K,ldw", [(8, 4, 5, 16), (7, 3, 6, 8), (5, 1, 4, 8), (3, 8, 9, 24)])
def test_host_offset_equals_the_oracle_layout(L, d, K, ldw):
    for layer in range(L):
        for ch in range(K):
            assert afx.afx_swap_host_offset(L, d, K, ldw, layer, ch) == oracle.group_layout_offset(layer, ch, L, d, K, ldw)
    for bad in ((L, 0), (-1, 0), (0, K), (0, -1)):
        with pytest.raises(afx.AfxError):
            afx.afx_swap_host_offset(L, d, K, ldw, *bad)


def test_pack_host_equals_the_oracle_packer():
    L, d, K, ldw = 5, 2, 7, 16
    per_layer = [np.ascontiguousarray(synth.normal_bits(11, l, (K, ldw), 1.0, "bf16")) for l in range(L)]
    out = np.zeros(L * K * ldw, np.uint16)
    afx.afx_swap_pack_host([a.ctypes.data for a in per_layer], L, d, K, ldw, out.ctypes.data)
    assert np.array_equal(out, oracle.pack_group_layout(per_layer, d))


def test_swap_descriptor_is_validated_on_the_host():
    FAKE = 0x7F0000000000
    ok = dict(dtype=1, n_layers=4, group=2, K=64, N=32, ldw=32, rows_pred=8, rows_miss=8, host_base=FAKE, dev_rows=FAKE)
    assert afx.afx_swap_device_bytes(afx.SwapDesc(**ok)) == 2 * 2 * 16 * 32 * 2

    def status(**kw):
        with pytest.raises(afx.AfxError) as e:
            afx.afx_swap_create(afx.SwapDesc(**{**ok, **kw}))
        return e.value.status

    assert status(dtype=5) == 4
    assert status(group=0) == 1 and status(K=0) == 1 and status(ldw=24) == 1 and status(host_base=None) == 1
    assert status(rows_pred=0, rows_miss=0) == 1
    assert status(N=36, ldw=40) == 2 and status(dev_rows=FAKE + 8) == 2

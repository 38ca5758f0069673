"""Pins for the oracle's cross-layer-group layout and preload bookkeeping (CPU only)."""
import numpy as np

import oracle
from paper_2504_08378_b200 import synth


def test_group_layout_is_the_papers_example():
    """Sec. 3 "Data layout": W_q of a 4-layer group N..N+3 is stored as
    [Ch0_N, Ch0_N+1, Ch0_N+2, Ch0_N+3, Ch1_N, Ch1_N+1, Ch1_N+2, Ch1_N+3, ..]."""
    L, d, K, ldw = 8, 4, 5, 16
    for first in (0, 4):  # both groups of an 8-layer stack
        want = [(ch, first + i) for ch in range(K) for i in range(4)]  # the paper's order
        offs = [oracle.group_layout_offset(layer, ch, L, d, K, ldw) for ch, layer in want]
        base = first * K * ldw
        assert offs == [base + n * ldw for n in range(K * 4)]


def test_group_layout_is_a_bijection_with_a_short_last_group():
    L, d, K, ldw = 7, 3, 6, 8   # groups {0,1,2}, {3,4,5}, {6}
    offs = sorted(oracle.group_layout_offset(l, j, L, d, K, ldw) for l in range(L) for j in range(K))
    assert offs == [n * ldw for n in range(L * K)]
    # a channel's columns of one group are adjacent: one read fetches all of them
    assert [oracle.group_layout_offset(l, 4, L, d, K, ldw) for l in (3, 4, 5)] == \
        [(3 * K + 4 * 3 + i) * ldw for i in range(3)]
    assert oracle.group_layout_offset(6, 2, L, d, K, ldw) == (6 * K + 2) * ldw  # the last group has one layer


def test_pack_group_layout_moves_every_column_to_its_offset():
    L, d, K, ldw = 5, 2, 7, 8
    per_layer = [synth.normal_bits(9, l, (K, ldw), 1.0, "bf16") for l in range(L)]
    img = oracle.pack_group_layout(per_layer, d)
    assert img.size == L * K * ldw
    for l in range(L):
        for j in range(K):
            o = oracle.group_layout_offset(l, j, L, d, K, ldw)
            assert np.array_equal(img[o:o + ldw], per_layer[l][j])
    # group {2,3}: channel 3 of both layers is one contiguous run
    o = oracle.group_layout_offset(2, 3, L, d, K, ldw)
    assert np.array_equal(img[o:o + 2 * ldw], np.concatenate([per_layer[2][3], per_layer[3][3]]))


def test_swap_acquire_hand_case():
    """P = [1,2,5,6] preloaded into rows 0..3; A = [1,5,6,7]: three found (rows 0, 2, 3), channel 7
    loaded on demand into the first on-demand row (the K = 8 cross-layer case worked by hand)."""
    out = oracle.swap_acquire([1, 2, 5, 6], [1, 5, 6, 7], rows_pred=4, rows_miss=2)
    assert out["slot"].tolist() == [0, 2, 3, 4] and out["ondemand"].tolist() == [7]
    assert (out["hits"], out["overflow"]) == (3, 0)
    # nothing predicted (the first layer group): everything is on demand, in list order
    out = oracle.swap_acquire([], [1, 5, 6, 7], rows_pred=4, rows_miss=4)
    assert out["slot"].tolist() == [4, 5, 6, 7] and out["hits"] == 0
    # on-demand rows run out: the rest is reported, not placed
    out = oracle.swap_acquire([1], [0, 1, 2, 3], rows_pred=2, rows_miss=2)
    assert out["slot"].tolist() == [2, 0, 3, -1] and out["overflow"] == 1 and out["ondemand"].tolist() == [0, 2]
    # a prediction longer than its rows: only the first rows_pred channels were preloaded
    out = oracle.swap_acquire([1, 2, 5, 6], [5, 6], rows_pred=3, rows_miss=2)
    assert out["slot"].tolist() == [2, 3] and out["ondemand"].tolist() == [6]


def test_swap_acquire_invariants_on_random_sets():
    g = synth.rng(10, 1)
    for _ in range(50):
        K = int(g.integers(8, 200))
        P = np.sort(g.choice(K, int(g.integers(0, K)), replace=False))
        A = np.sort(g.choice(K, int(g.integers(0, K)), replace=False))
        rp, rm = int(g.integers(1, K + 1)), int(g.integers(0, K + 1))
        out = oracle.swap_acquire(P, A, rp, rm)
        placed = out["slot"][out["slot"] >= 0]
        assert len(set(placed.tolist())) == placed.size                   # no row serves two channels
        assert out["hits"] == np.intersect1d(A, P[:rp]).size              # exactly the preloaded ones hit
        assert out["hits"] + out["ondemand"].size + out["overflow"] == A.size
        assert np.array_equal(out["ondemand"], np.setdiff1d(A, P[:rp])[: out["ondemand"].size])
        assert out["ondemand"].size == min(rm, A.size - out["hits"])

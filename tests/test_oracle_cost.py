"""Pins for the oracle's cost model (Sec. 4.1, Eq. 1-9): numbers worked by hand, and the
behaviour the text states."""
import pytest

import oracle


def test_cost_model_hand_numbers():
    """S_l = 400 MB, sp = 0.5, N = 4 -> M_cl = 800 MB (Eq. 9).  hr = 0.5, si = 0.8, BW_mem 50 GB/s,
    flash 0.5 GB/s small / 2 GB/s large:
      T_load = 800e6 * 0.5 / 0.5e9 = 0.8 s (Eq. 3);  T_comp = 800e6 / 50e9 = 0.016 s (Eq. 4);
      T_onload = 400e6 * 0.5 * 0.5 * 0.2 / 0.5e9 = 0.04 s (Eq. 6);  T_preload = 400e6 / 2e9 = 0.2 s (Eq. 7);
      T_overlap = 0.04 + max(0.2, 0.016) = 0.24 s (Eq. 5);  T_decode = 0.8 + 0.24 + 0.016 = 1.056 s (Eq. 1);
      M = 800 MB + 1 GB cache + 0.25 GB KV = 2.05 GB (Eq. 8)."""
    c = oracle.cost_model(sp=0.5, hr=0.5, si=0.8, N=4, S_l=400e6, bw_mem=50e9, bw_flash_small=0.5e9,
                          bw_flash_large=2e9, M_cache=1e9, M_kv=0.25e9, n_layers=32)
    want = dict(M_cl=800e6, M=2.05e9, T_load=0.8, T_comp=0.016, T_onload=0.04, T_preload=0.2, T_overlap=0.24,
                T_decode=1.056, T_token=0.8 + 7 * 0.24 + 0.016)
    for k, v in want.items():
        assert c[k] == pytest.approx(v, rel=1e-12), k


def test_cost_model_limits():
    base = dict(sp=0.6, si=0.8, N=2, S_l=400e6, bw_mem=50e9, bw_flash_small=1e9, bw_flash_large=3e9)
    # a cache that always hits removes every flash term: decoding is two group computations
    c = oracle.cost_model(hr=1.0, **base)
    assert c["T_load"] == 0 and c["T_onload"] == 0 and c["T_preload"] == 0
    assert c["T_decode"] == pytest.approx(2 * c["T_comp"])
    # perfect cross-layer similarity leaves nothing to load on demand
    assert oracle.cost_model(hr=0.3, **{**base, "si": 1.0})["T_onload"] == 0
    # when preloading is the slower side it, not the computation, sets the overlap stage
    c = oracle.cost_model(hr=0.0, **base)
    assert c["T_preload"] > c["T_comp"] and c["T_overlap"] == pytest.approx(c["T_onload"] + c["T_preload"])
    # a denser model costs proportionally more of everything
    a, b = oracle.cost_model(hr=0.2, **base), oracle.cost_model(hr=0.2, **{**base, "sp": 0.2})
    assert b["T_decode"] == pytest.approx(2 * a["T_decode"]) and b["M_cl"] == pytest.approx(2 * a["M_cl"])

"""The library's cost model (host arithmetic, no GPU) against the oracle's Eq. 1-9, and the
greedy search against cases whose answer follows from the rule in Sec. 4.1."""
import pytest

import oracle
from paper_2504_08378_b200 import afx

STOP = dict(balanced=0, gain=1, memory=2, n_max=3)


@pytest.mark.parametrize("kw", [
    dict(sp=0.5, hr=0.5, si=0.8, N=4, n_layers=32, S_l=400e6, bw_mem=50e9, bw_flash_small=0.5e9, bw_flash_large=2e9,
         M_cache=1e9, M_kv=0.25e9),
    dict(sp=0.6, hr=0.0, si=0.3, N=1, n_layers=8, S_l=1.7e9, bw_mem=6.4e12, bw_flash_small=50e9, bw_flash_large=51e9,
         M_cache=0.0, M_kv=0.0),
    dict(sp=0.0, hr=1.0, si=1.0, N=7, n_layers=30, S_l=1e8, bw_mem=1e10, bw_flash_small=1e8, bw_flash_large=1e9,
         M_cache=5e8, M_kv=1e8),
])
def test_cost_eval_equals_the_oracle(kw):
    got = afx.afx_cost_eval(**kw)
    okw = {k: v for k, v in kw.items()}
    want = oracle.cost_model(**okw)
    for name, v in want.items():
        assert got[name] == pytest.approx(v, rel=1e-12, abs=0.0), name


def test_cost_eval_rejects_bad_parameters():
    ok = dict(sp=0.5, hr=0.5, si=0.8, N=4, n_layers=32, S_l=4e8, bw_mem=5e10, bw_flash_small=5e8, bw_flash_large=2e9)
    for bad in (dict(sp=1.5), dict(hr=-0.1), dict(N=0), dict(bw_mem=0.0), dict(S_l=float("nan"))):
        with pytest.raises(afx.AfxError):
            afx.afx_cost_eval(**{**ok, **bad})


def base_search(**over):
    kw = dict(S_m=32 * 400e6, S_l=400e6, n_layers=32, M_max=0.5 * 32 * 400e6, M_kv=0.2e9, bw_mem=50e9,
              bw_flash_small=0.3e9, column_bytes=16384.0, si=0.8, min_gain=0.05, N_max=8)
    kw.update(over)
    return kw


def test_search_sets_sparsity_from_the_budget_and_gives_the_rest_to_the_cache():
    chunk = [(16384, 0.5e9), (65536, 2e9)]       # a phone-like flash: 4 x larger reads run 4 x faster
    hr = [(0.0, 0.0), (0.5, 0.8)]
    r = afx.afx_cost_search(chunk, hr, **base_search())
    assert r["sp"] == pytest.approx(0.5)         # sp = 1 - M_max / S_m
    M_cl = 400e6 * 0.5 * r["N"]
    assert r["M_cache"] == pytest.approx(0.5 * 32 * 400e6 - 0.2e9 - M_cl)
    assert r["hr"] == pytest.approx(0.8 * (r["M_cache"] / (32 * 400e6)) / 0.5)
    want = oracle.cost_model(sp=r["sp"], hr=r["hr"], si=0.8, N=r["N"], S_l=400e6, bw_mem=50e9, bw_flash_small=0.3e9,
                             bw_flash_large=r["bw_flash_large"], M_cache=r["M_cache"], M_kv=0.2e9, n_layers=32)
    for name, v in want.items():
        assert r["cost"][name] == pytest.approx(v, rel=1e-12)
    # the read bandwidth saturates at 4 layers per group (64 KB chunks): the 5th layer gains nothing
    assert r["N"] == 4 and r["stop_reason"] == STOP["gain"]


def test_search_stops_at_once_when_chunk_size_does_not_matter():
    """A link whose throughput does not depend on the read size (what a GPU's host link shows):
    a second layer per group lowers nothing, so the group stays at one layer."""
    r = afx.afx_cost_search([(2048, 51e9), (1 << 20, 51e9)], [(0.0, 0.0), (0.3, 0.5)], **base_search(bw_flash_small=51e9, bw_mem=6.4e12))
    assert r["N"] == 1 and r["stop_reason"] == STOP["gain"]


def test_search_stops_when_preloading_hides_behind_computation():
    r = afx.afx_cost_search([(16384, 100e9), (65536, 200e9)], [(0.0, 0.0), (0.5, 0.8)], **base_search(bw_mem=20e9))
    assert r["stop_reason"] == STOP["balanced"] and r["N"] == 1
    assert r["cost"]["T_preload"] <= r["cost"]["T_comp"]


def test_search_respects_the_memory_budget():
    # budget = 10 % of the model, most of it KV cache: groups of more than 2 layers do not fit
    kw = base_search(M_max=0.1 * 32 * 400e6, M_kv=0.1 * 32 * 400e6 - 100e6, min_gain=0.0)
    r = afx.afx_cost_search([(16384, 0.5e9), (1 << 20, 8e9)], [(0.0, 0.0), (0.5, 0.8)], **kw)
    assert r["sp"] == pytest.approx(0.9) and r["N"] == 2 and r["stop_reason"] == STOP["memory"]
    with pytest.raises(afx.AfxError) as e:
        afx.afx_cost_search([(16384, 0.5e9)], [(0.0, 0.0)], **base_search(M_max=1e9, M_kv=0.999e9))
    assert e.value.status == 3

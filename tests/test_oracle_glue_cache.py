"""Pins for the decoder-layer glue (against torch fp64 library routines) and the LFU cache
(the paper's worked example, a pure-Python brute force, invariants)."""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2504_08378_b200 import synth


def _ulp_diff(a_bits, b_bits):
    """distance in representable values between two same-sign 16-bit patterns"""
    a = a_bits.astype(np.int32)
    b = b_bits.astype(np.int32)
    return np.abs(a - b)


@pytest.mark.parametrize("dt,tdt", [("f16", torch.float16), ("bf16", torch.bfloat16)])
def test_rmsnorm_matches_torch(dt, tdt):
    g = np.random.default_rng(1)
    h = g.standard_normal((3, 512)) * 3.0
    gain = 1.0 + 0.1 * g.standard_normal(512)
    got = oracle.rmsnorm(h, gain, 1e-5, dt)
    ht = torch.from_numpy(h)
    want = torch.nn.functional.rms_norm(ht, (512,), torch.from_numpy(gain), 1e-5)
    want_bits = want.to(tdt).view(torch.int16).numpy().view(np.uint16)
    assert (_ulp_diff(got, want_bits) <= 1).all()        # torch rounds fp64 -> fp32 -> 16 bit
    assert (got == want_bits).mean() > 0.99


def test_rope_matches_complex_rotation():
    g = np.random.default_rng(2)
    T, heads, D = 2, 3, 128
    v = g.standard_normal((T, heads, D))
    pos = np.array([5, 2048], np.int32)
    got = oracle.rope(v, pos, 10000.0)
    z = v[..., 0::2] + 1j * v[..., 1::2]
    freqs = 10000.0 ** (-np.arange(0, D, 2) / D)
    rot = np.exp(1j * pos[:, None, None] * freqs[None, None, :])
    w = z * rot
    want = np.empty_like(v)
    want[..., 0::2], want[..., 1::2] = w.real, w.imag
    assert np.allclose(got, want, rtol=0, atol=1e-12)
    assert np.allclose(np.linalg.norm(got, axis=-1), np.linalg.norm(v, axis=-1))
    assert np.array_equal(oracle.rope(v, np.zeros(T, np.int32)), v)     # position 0: identity


@pytest.mark.parametrize("q_heads,kv_heads", [(4, 4), (8, 2)])
def test_attention_matches_torch_sdpa(q_heads, kv_heads):
    g = np.random.default_rng(3)
    L, D = 37, 128
    q = g.standard_normal((q_heads, D))
    kc = synth.normal_bits(4, 1, (L + 3, kv_heads, D), 1.0, "f16")
    vc = synth.normal_bits(4, 2, (L + 3, kv_heads, D), 1.0, "f16")
    got = oracle.attention(q, kc, vc, L, "f16")
    k = torch.from_numpy(synth.bits_to_f32(kc[:L], "f16")).double().permute(1, 0, 2)
    v = torch.from_numpy(synth.bits_to_f32(vc[:L], "f16")).double().permute(1, 0, 2)
    rep = q_heads // kv_heads
    k, v = k.repeat_interleave(rep, 0), v.repeat_interleave(rep, 0)
    out = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[:, None, :], k, v)[:, 0, :]
    want = out.to(torch.float16).view(torch.int16).numpy().view(np.uint16)
    assert (_ulp_diff(got, want) <= 1).all()
    assert (got == want).mean() > 0.99


def test_silu_mul_matches_torch():
    g = np.random.default_rng(4)
    a, b = g.standard_normal(4000) * 3, g.standard_normal(4000)
    got = oracle.silu_mul(a, b, "bf16")
    want = (torch.nn.functional.silu(torch.from_numpy(a)) * torch.from_numpy(b))
    want = want.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (_ulp_diff(got, want) <= 1).all() and (got == want).mean() > 0.99


# ------------------------------------------------------------------ cache

def test_paper_cache_example(golden_dir):
    with open(os.path.join(golden_dir, "cache_example.json")) as f:
        ex = json.load(f)
    for initial in (ex["initial"], [0, 2, 3, 5]):
        c = oracle.LfuCache(ex["K"], ex["capacity"])
        c.reset_counts()
        c.install(initial)
        for tok in ex["tokens"]:
            before = set(c.cached().tolist())
            r = c.step(tok["active"])
            assert (r["hits"], r["misses"]) == (tok["hits"], tok["misses"])
            assert r["hits"] / (r["hits"] + r["misses"]) == tok["hit_ratio"]
            assert c.cached().tolist() == tok["cached_after"]
            if "replaced" in tok:
                assert before - set(c.cached().tolist()) == {tok["replaced"]}


def _python_lfu(K, C, steps, initial=()):
    """Independent pure-Python restatement with dicts (brute force on tiny inputs)."""
    where, freq, free = {}, [0] * K, list(range(C))
    for j in initial:
        where[j] = free.pop(0)
    log = []
    for act in steps:
        for j in act:
            freq[j] += 1
        hits = misses = trans = 0
        slots = []
        for j in act:
            if j in where:
                hits += 1
                slots.append(where[j])
                continue
            misses += 1
            if free:
                where[j] = min(free)
                free.remove(where[j])
                slots.append(where[j])
                continue
            cand = [(freq[v], v) for v in where if v not in act]
            if cand and freq[j] >= min(cand)[0]:
                v = min(cand)[1]
                where[j] = where.pop(v)
                slots.append(where[j])
            else:
                slots.append(C + trans)
                trans += 1
        log.append((hits, misses, trans, slots, sorted(where)))
    return log


@pytest.mark.parametrize("K,C,k", [(8, 4, 4), (24, 6, 10), (40, 40, 12), (30, 1, 3)])
def test_cache_matches_python_brute_force(K, C, k):
    g = np.random.default_rng(K * 100 + C)
    w = 1.0 / np.arange(1, K + 1) ** 1.1
    steps = [sorted(g.choice(K, k, replace=False, p=w / w.sum()).tolist()) for _ in range(40)]
    want = _python_lfu(K, C, steps)
    c = oracle.LfuCache(K, C)
    for act, (hits, misses, trans, slots, cached) in zip(steps, want):
        r = c.step(act)
        assert (r["hits"], r["misses"], r["transients"]) == (hits, misses, trans)
        assert r["slot"].tolist() == slots
        assert c.cached().tolist() == cached
        # invariants: slot map is a bijection between cached channels and used slots
        used = c.chan_of[c.chan_of >= 0]
        assert len(set(used.tolist())) == used.size <= C
        assert all(c.slot_of[c.chan_of[s]] == s for s in range(C) if c.chan_of[s] >= 0)
        assert r["hits"] + r["misses"] == len(act)


def test_cache_as_large_as_the_tensor_misses_each_channel_once():
    K = 64
    g = np.random.default_rng(9)
    c = oracle.LfuCache(K, K)
    seen, total_miss = set(), 0
    for _ in range(30):
        act = np.sort(g.choice(K, 20, replace=False))
        r = c.step(act)
        assert r["misses"] == len(set(act.tolist()) - seen) and r["transients"] == 0
        seen |= set(act.tolist())
        total_miss += r["misses"]
    assert total_miss == len(seen)

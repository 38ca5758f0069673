"""Pins for the oracle's 16-bit format code against numpy (fp16) and torch (bf16)."""
import numpy as np
import torch

import oracle


def test_decode_f16_all_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    got = oracle.decode(bits, "f16")
    want = bits.view(np.float16).astype(np.float64)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])
    assert np.array_equal(np.signbit(got[ok]), np.signbit(want[ok]))


def test_decode_bf16_all_patterns_match_torch():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    got = oracle.decode(bits, "bf16")
    want = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])


def _probe_values():
    g = np.random.default_rng(7)
    v = np.concatenate([
        g.standard_normal(20000) * 10.0 ** g.integers(-9, 6, 20000),
        g.standard_normal(2000) * 1e-42,            # bf16 subnormal range
        np.array([0.0, -0.0, 1.0, -1.0, 65504.0, 65519.9, 65520.0, 1e39, -1e39, np.inf, -np.inf,
                  2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -25, 2.0 ** -14, 1.0 + 2.0 ** -11,
                  1.0 + 3 * 2.0 ** -11, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8]),
    ])
    return v


def test_round_f16_matches_numpy_rne():
    # float64 -> float16 in numpy is a single correctly rounded conversion
    v = _probe_values()
    got = oracle.round_to(v, "f16")
    with np.errstate(over="ignore"):
        want = v.astype(np.float16).view(np.uint16)
    assert np.array_equal(got, want)


def test_round_bf16_matches_torch_rne_on_float32_inputs():
    # torch rounds float32 -> bfloat16 to nearest-even; feed float32-representable values so
    # that the oracle's single fp64 rounding and torch's fp32 rounding see the same number
    v = _probe_values().astype(np.float32)
    v = v[np.isfinite(v) | np.isinf(v)]
    got = oracle.round_to(v.astype(np.float64), "bf16")
    want = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)


def test_round_then_decode_is_identity_on_representable_values():
    for dt in ("f16", "bf16"):
        bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
        vals = oracle.decode(bits, dt)
        ok = ~np.isnan(vals)
        assert np.array_equal(oracle.round_to(vals[ok], dt), bits[ok])


def test_synth_bits_agree_with_oracle_decode():
    from paper_2504_08378_b200 import synth
    for dt in ("f16", "bf16"):
        b = synth.laplace_bits(3, 1, (4096,), dt)
        assert np.array_equal(oracle.decode(b, dt), synth.bits_to_f32(b, dt).astype(np.float64))

"""Pins for the oracle's Q16 / Q32 emulation (Sec. 2: float16 1-5-10, bfloat16 1-8-7; Sec. 4: round to nearest)."""
import numpy as np
import torch

from oracle.quantize import quantize, max_finite, precision_bits


def test_unit_roundoffs_match_paper():
    # Sec. 3: u_L = 2^-11 for float16 and 2^-8 for bfloat16
    assert precision_bits("f16") == 11 and precision_bits("bf16") == 8 and precision_bits("f32") == 24


def test_f16_all_bit_patterns_are_fixed_points():
    h = np.arange(65536, dtype=np.uint16).view(np.float16)
    x = h.astype(np.float64)
    qx = quantize(x, "f16")
    fin = np.isfinite(x)
    assert np.array_equal(qx[fin], x[fin])
    assert np.all(np.isnan(qx[np.isnan(x)]))
    assert np.array_equal(qx[np.isinf(x)], x[np.isinf(x)])


def test_bf16_all_bit_patterns_are_fixed_points():
    bits = (np.arange(65536, dtype=np.uint32) << 16).view(np.float32)
    x = bits.astype(np.float64)
    fin = np.isfinite(x)
    assert np.array_equal(quantize(x, "bf16")[fin], x[fin])


def test_f16_matches_numpy_half_conversion():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.standard_normal(200000) * np.exp(rng.uniform(-20, 12, 200000)),
        rng.uniform(-2 ** -14, 2 ** -14, 50000),          # subnormal range
        rng.uniform(65000, 66000, 20000),                  # overflow edge
    ])
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).astype(np.float64)      # numpy rounds double -> half correctly
    assert np.array_equal(quantize(x, "f16"), ref)


def test_f32_matches_numpy_single_conversion():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(100000) * np.exp(rng.uniform(-100, 80, 100000))
    assert np.array_equal(quantize(x, "f32"), x.astype(np.float32).astype(np.float64))


def test_bf16_matches_torch_conversion_on_fp32_inputs():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(300000) * np.exp(rng.uniform(-80, 80, 300000))).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(quantize(x.astype(np.float64), "bf16"), ref)


def test_ties_go_to_even_and_overflow_edge():
    # float16 spacing at 2048 is 2: 2049 is a tie -> 2048 (even mantissa), 2051 -> 2052
    assert quantize(2049.0, "f16") == 2048.0 and quantize(2051.0, "f16") == 2052.0
    assert quantize(2049.0000001, "f16") == 2050.0
    # largest finite 65504, spacing 32: 65520 is the tie with 2^16 -> Inf; just below stays finite
    assert max_finite("f16") == 65504.0
    assert np.isinf(quantize(65520.0, "f16")) and quantize(65519.999, "f16") == 65504.0
    assert quantize(-65520.0, "f16") == -np.inf
    # gradual underflow: smallest subnormal 2^-24; half of it ties to zero, a bit more rounds up
    assert quantize(2.0 ** -25, "f16") == 0.0 and quantize(2.0 ** -25 * 1.0001, "f16") == 2.0 ** -24
    assert quantize(3 * 2.0 ** -25, "f16") == 2.0 ** -23      # tie between 1 and 2 ulps -> even (2)
    # bfloat16: 8 significant bits, spacing at 256 is 2
    assert quantize(257.0, "bf16") == 256.0 and quantize(259.0, "bf16") == 260.0
    assert np.isnan(quantize(np.nan, "bf16"))
    assert quantize(1e39, "bf16") == np.inf and quantize(3.0e38, "bf16") < np.inf


def test_direct_rounding_not_double_rounding():
    # 1 + 2^-8 + 2^-30 lies just above the bf16 tie at 1 + 2^-8: it must round up to 1 + 2^-7,
    # whereas rounding to fp32 first would land on the tie and go to even (1.0).
    x = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert quantize(x, "bf16") == 1.0 + 2.0 ** -7
    assert quantize(float(np.float32(x)), "bf16") == 1.0


def test_relative_error_bound():
    rng = np.random.default_rng(3)
    x = rng.standard_normal(100000) * 100
    for fmt in ("f16", "bf16", "f32"):
        r = np.abs(quantize(x, fmt) - x) / np.abs(x)
        assert r.max() <= 2.0 ** -precision_bits(fmt)

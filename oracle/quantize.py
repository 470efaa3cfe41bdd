"""Quantisation operators Q16 / Q32 of Sec. 2 ("Mixed Precision Training"), emulated in fp64.

TEST INFRASTRUCTURE ONLY: a slow CPU statement of the paper's rounding, used by
the tests, the smoke check and the benchmark's CPU-baseline leg.  It shares no
code with the CUDA path.

Q16 maps to the representable numbers of float16 (1 sign, 5 exponent, 10
mantissa bits) or bfloat16 (1-8-7); Q32 to float32 (1-8-23).  Rounding is
round-to-nearest, ties to even (Sec. 4: "round-to-nearest mode, the IEEE 754
default"), applied directly to the wide (fp64) value: values beyond the
largest finite number by half an ulp or more become +-Inf, subnormals are
kept (gradual underflow), NaN stays NaN.

Unit roundoffs (Sec. 3): u_L = 2^-11 for float16, 2^-8 for bfloat16; 2^-24
for float32.  `precision_bits` is p with u = 2^-p.
"""
from __future__ import annotations

import numpy as np

# name -> (explicit mantissa bits t, minimum normal exponent emin, maximum exponent emax)
FORMATS = {
    "f16": (10, -14, 15),
    "bf16": (7, -126, 127),
    "f32": (23, -126, 127),
}


def precision_bits(fmt: str) -> int:
    """p such that the unit roundoff is 2^-p (p = t + 1)."""
    if fmt == "f64":
        return 53
    return FORMATS[fmt][0] + 1


def max_finite(fmt: str) -> float:
    t, _, emax = FORMATS[fmt]
    return float((2.0 - 2.0 ** (-t)) * 2.0 ** emax)


def quantize(x, fmt: str) -> np.ndarray:
    """Round fp64 values to format `fmt` (result returned as fp64).  "f64" is the identity.

    |x| = m * 2^e with m in [0.5, 1): the spacing of the target format around
    x is 2^q with q = max(e - p, emin - t); x is rounded to a multiple of 2^q
    by rint (ties to even); a result above the largest finite value is Inf.
    """
    x = np.asarray(x, dtype=np.float64)
    if fmt == "f64":
        return x
    t, emin, _ = FORMATS[fmt]
    p = t + 1
    ax = np.abs(x)
    finite = np.isfinite(ax)
    axf = np.where(finite, ax, 0.0)
    _, e = np.frexp(axf)
    q = np.maximum(e - p, emin - t).astype(np.int64)
    # axf * 2^-q is at most 2^p and at least 0: exact scaling by a power of two
    r = np.ldexp(np.rint(np.ldexp(axf, -q)), q)
    r = np.where(r > max_finite(fmt), np.inf, r)
    r = np.where(finite, r, ax)  # Inf stays Inf, NaN stays NaN
    return np.copysign(r, x)


def is_nonfinite_any(x) -> bool:
    return not bool(np.all(np.isfinite(x)))

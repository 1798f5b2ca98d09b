"""Floating-point formats and the quantiser q(.) (test infrastructure, fp64 NumPy).

Follows the paper's section "Floating-point formats for deep learning"
(Definition paragraph: sign / exponent / mantissa fields, bias = 2^(E-1) - 1,
value = (-1)^s * 2^exponent * (1 + mant / 2^M), plus subnormals and special
values) and the "Quantisation error" paragraph (q maps an input to the nearest
representable value; out-of-range inputs incur clipping, i.e. saturation).
The FP8 variants are the "(b)" rows of the appendix table "Common floating
point formats for deep learning" (E4: max exp 8, min exp -6; E5: max exp 15,
min exp -14), which are the OCP E4M3 / E5M2 formats.

Readings taken where the paper leaves the choice open:
  * ties go to the neighbour whose mantissa code is even;
  * FP8 overflow (including +-Inf) saturates to the largest finite value,
    NaN stays NaN;
  * FP16 / BFLOAT16 follow IEEE 754 (overflow rounds to +-Inf).

Every function works on float64 arrays; float32 inputs are widened exactly.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Format:
    """A binary floating-point format with E exponent bits and M mantissa bits."""

    name: str
    E: int                # exponent bits
    M: int                # mantissa bits
    bias: int             # exponent bias, 2^(E-1) - 1 for all formats used here
    max_exp: int          # largest exponent of a finite value ("Max exp." column)
    max_mant: int         # largest mantissa code at max_exp that is still finite
    saturate: bool        # True: overflow clips to +-max finite; False: IEEE (+-Inf)
    has_inf: bool         # whether the code space contains +-Inf

    @property
    def min_exp(self) -> int:
        """Smallest exponent of a normal value ("Min exp." column)."""
        return 1 - self.bias

    @property
    def max_finite(self) -> float:
        return float(2.0 ** self.max_exp * (1.0 + self.max_mant / 2.0 ** self.M))

    @property
    def min_normal(self) -> float:
        return float(2.0 ** self.min_exp)

    @property
    def min_subnormal(self) -> float:
        return float(2.0 ** (self.min_exp - self.M))

    @property
    def bits(self) -> int:
        return 1 + self.E + self.M


# E4 "(b)": bias 7; the all-ones exponent is an ordinary binade (max exp 8) whose
# last mantissa code is the only NaN, so the largest finite value is 2^8 * 1.75.
E4M3 = Format("e4m3", E=4, M=3, bias=7, max_exp=8, max_mant=6, saturate=True, has_inf=False)
# E5 "(b)": IEEE-like, all-ones exponent reserved for Inf / NaN.
E5M2 = Format("e5m2", E=5, M=2, bias=15, max_exp=15, max_mant=3, saturate=True, has_inf=True)
FP16 = Format("fp16", E=5, M=10, bias=15, max_exp=15, max_mant=1023, saturate=False, has_inf=True)
BF16 = Format("bf16", E=8, M=7, bias=127, max_exp=127, max_mant=127, saturate=False, has_inf=True)

FORMATS = {f.name: f for f in (E4M3, E5M2, FP16, BF16)}


def quantise(x, fmt: Format) -> np.ndarray:
    """q(x): the value of `fmt` nearest to each element of x, as float64.

    Steps, for finite x: pick the binade exponent e = floor(log2 |x|), clamped
    below at the format's minimum normal exponent (subnormals share that
    spacing); the representable values around x are multiples of the spacing
    2^(e-M); round x / spacing to the nearest integer with ties to even (the
    integer's parity is the mantissa code's parity); then apply the overflow
    rule of the format.
    """
    x = np.asarray(x, dtype=np.float64)
    out = np.empty_like(x)
    nan = np.isnan(x)
    a = np.abs(np.where(nan, 0.0, x))
    finite = np.isfinite(a)
    af = np.where(finite, a, 0.0)
    # frexp: af = m * 2^ex with m in [0.5, 1)  =>  floor(log2 af) = ex - 1
    _, ex = np.frexp(af)
    e = np.maximum(ex.astype(np.int64) - 1, fmt.min_exp)
    spacing = np.ldexp(1.0, (e - fmt.M).astype(np.int64))
    r = np.rint(af / spacing) * spacing          # exact: spacing is a power of two
    if fmt.saturate:
        r = np.where(finite, np.minimum(r, fmt.max_finite), fmt.max_finite)
    else:
        # IEEE: a rounded magnitude beyond the largest finite value becomes Inf
        r = np.where(finite & (r <= fmt.max_finite), r, np.inf)
    out = np.copysign(r, np.where(nan, 1.0, x))
    out = np.where(nan, np.nan, out)
    return out


def encode(v, fmt: Format) -> np.ndarray:
    """Bit pattern (unsigned integer array) of values that are already representable."""
    v = np.asarray(v, dtype=np.float64)
    sign = np.signbit(v).astype(np.uint32)
    a = np.abs(v)
    nan = np.isnan(v)
    inf = np.isinf(v)
    af = np.where(nan | inf, 0.0, a)
    _, ex = np.frexp(af)
    e = ex.astype(np.int64) - 1
    normal = af >= fmt.min_normal
    e = np.where(normal, e, fmt.min_exp)
    frac = af / np.ldexp(1.0, e)                   # in [1,2) for normals, [0,1) for subnormals
    mant = np.rint((frac - np.where(normal, 1.0, 0.0)) * 2.0 ** fmt.M).astype(np.int64)
    bexp = np.where(normal, e + fmt.bias, 0).astype(np.int64)
    all_ones = (1 << fmt.E) - 1
    if fmt.has_inf:
        bexp = np.where(inf, all_ones, bexp)
        mant = np.where(inf, 0, mant)
        bexp = np.where(nan, all_ones, bexp)
        mant = np.where(nan, (1 << fmt.M) - 1, mant)
    else:
        if np.any(inf):
            raise ValueError(f"{fmt.name} has no infinity")
        bexp = np.where(nan, all_ones, bexp)
        mant = np.where(nan, (1 << fmt.M) - 1, mant)
    code = (sign.astype(np.int64) << (fmt.E + fmt.M)) | (bexp << fmt.M) | mant
    dtype = np.uint8 if fmt.bits == 8 else np.uint16
    return code.astype(dtype)


def decode(code, fmt: Format) -> np.ndarray:
    """Value (float64) of each bit pattern, straight from the format definition."""
    c = np.asarray(code).astype(np.int64)
    s = (c >> (fmt.E + fmt.M)) & 1
    bexp = (c >> fmt.M) & ((1 << fmt.E) - 1)
    mant = c & ((1 << fmt.M) - 1)
    normal = bexp > 0
    val = np.where(
        normal,
        np.ldexp(1.0 + mant / 2.0 ** fmt.M, (bexp - fmt.bias).astype(np.int64)),
        np.ldexp(mant / 2.0 ** fmt.M, fmt.min_exp),
    )
    all_ones = (1 << fmt.E) - 1
    if fmt.has_inf:
        val = np.where((bexp == all_ones) & (mant == 0), np.inf, val)
        val = np.where((bexp == all_ones) & (mant != 0), np.nan, val)
    else:
        val = np.where((bexp == all_ones) & (mant == (1 << fmt.M) - 1), np.nan, val)
    return np.where(s == 1, -val, val)


def quantise_codes(x, fmt: Format) -> np.ndarray:
    """Bit patterns of q(x)."""
    return encode(quantise(x, fmt), fmt)


def scaled_cast(x, scale, fmt: Format) -> np.ndarray:
    """Codes of q(s * x) where the product is formed in float32 first.

    The cast op multiplies by its scale once, in single precision, and rounds the
    float32 product once to the target format.  `x` may be float32 or a 16-bit
    float array (widened exactly).
    """
    xf = np.asarray(x).astype(np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        prod = xf * np.float32(scale)
    return quantise_codes(prod.astype(np.float64), fmt)


def snr(x, fmt: Format) -> float:
    """Signal-to-noise ratio E[X^2] / E[(q(X) - X)^2] of the quantiser on samples x."""
    x = np.asarray(x, dtype=np.float64)
    err = quantise(x, fmt) - x
    return float(np.mean(x * x) / np.mean(err * err))


def exponent_histogram(x, exp_lo: int, nbins: int) -> np.ndarray:
    """Counts of floor(log2 |x|) over the samples (appendix "Histograms of tensor-scaling within BERT":
    the figures plot exactly this for activations, weights and gradients).

    Returns nbins + 2 counts: [0] everything below 2^exp_lo (zeros included), [1 + k] the values with
    2^(exp_lo + k) <= |x| < 2^(exp_lo + k + 1), [nbins + 1] everything at or above 2^(exp_lo + nbins),
    infinities and NaNs."""
    a = np.abs(np.asarray(x, dtype=np.float64)).ravel()
    out = np.zeros(nbins + 2, dtype=np.int64)
    finite = np.isfinite(a)
    out[nbins + 1] += int((~finite).sum())
    a = a[finite]
    lo, hi = 2.0 ** exp_lo, 2.0 ** (exp_lo + nbins)
    out[0] += int((a < lo).sum())
    out[nbins + 1] += int((a >= hi).sum())
    mid = a[(a >= lo) & (a < hi)]
    _, e = np.frexp(mid)                       # mid = m * 2^e with 0.5 <= m < 1, so floor(log2 mid) = e - 1
    np.add.at(out, 1 + (e - 1 - exp_lo), 1)
    return out

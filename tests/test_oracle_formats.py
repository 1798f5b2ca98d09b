"""Pins for the oracle's quantiser: library decoders / casters, brute force, the paper's format table."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import formats as F
from tests.golden.load import load

GOLD = load("paper_constants.txt")
TORCH_FP8 = {"e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}


def torch_decode(fmt):
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    return codes.view(TORCH_FP8[fmt.name]).to(torch.float64).numpy()


@pytest.mark.parametrize("fmt", [F.E4M3, F.E5M2])
def test_decode_matches_library_tables(fmt):
    ours = F.decode(np.arange(256), fmt)
    lib = torch_decode(fmt)
    assert np.array_equal(np.isnan(ours), np.isnan(lib))
    ok = ~np.isnan(lib)
    assert np.array_equal(ours[ok], lib[ok])
    assert np.array_equal(np.signbit(ours[ok]), np.signbit(lib[ok]))


@pytest.mark.parametrize("name", ["fp16", "bf16", "e5m2", "e4m3"])
def test_format_table_exponent_limits(name):
    fmt = F.FORMATS[name]
    assert fmt.E == GOLD[f"{name}_E"] and fmt.M == GOLD[f"{name}_M"]
    assert fmt.max_exp == GOLD[f"{name}_max_exp"]
    assert fmt.min_exp == GOLD[f"{name}_min_exp"]
    assert fmt.bias == 2 ** (fmt.E - 1) - 1


def test_extreme_values():
    assert F.E4M3.max_finite == 448.0 and F.E4M3.min_normal == 2.0 ** -6 and F.E4M3.min_subnormal == 2.0 ** -9
    assert F.E5M2.max_finite == 57344.0 and F.E5M2.min_normal == 2.0 ** -14 and F.E5M2.min_subnormal == 2.0 ** -16
    assert F.FP16.max_finite == 65504.0


def brute_force_nearest(x, fmt):
    """Nearest finite table value; exact ties go to the even code; no overflow rule needed
    because clipping to the largest finite value *is* the nearest finite value."""
    table = torch_decode(fmt)
    codes = np.arange(256)
    keep = np.isfinite(table) & (codes < 128)            # non-negative finite values
    vals = [Fraction(float(v)) for v in table[keep]]     # exact rationals: no rounding in the search
    cds = codes[keep]
    out = np.empty(len(x), dtype=np.uint8)
    for i, xi in enumerate(x):
        a = abs(Fraction(float(xi)))
        d = [abs(v - a) for v in vals]
        dmin = min(d)
        best = [j for j, dj in enumerate(d) if dj == dmin]
        assert len(best) in (1, 2)
        c = cds[best[0]]
        if len(best) == 2 and c % 2 == 1:
            c = cds[best[1]]
        out[i] = c | (0x80 if np.signbit(xi) else 0)
    return out


def interesting_values(fmt, rng):
    table = torch_decode(fmt)
    pos = np.sort(table[np.isfinite(table) & (table >= 0)])
    mids = (pos[:-1] + pos[1:]) / 2
    near = np.concatenate([np.nextafter(mids.astype(np.float32), np.float32(np.inf)),
                           np.nextafter(mids.astype(np.float32), np.float32(-np.inf))]).astype(np.float64)
    rnd = rng.standard_normal(1500) * np.exp2(rng.integers(-20, 18, 1500))
    big = np.array([fmt.max_finite * 1.01, fmt.max_finite * 1.5, 1e30, 3.0e38])
    tiny = np.array([fmt.min_subnormal * t for t in (0.25, 0.49999, 0.5, 0.50001, 0.75, 1.0, 1.5, 2.5)])
    x = np.concatenate([pos, mids, near, rnd, big, tiny, [0.0]])
    x = x.astype(np.float32).astype(np.float64)
    return np.concatenate([x, -x])


@pytest.mark.parametrize("fmt", [F.E4M3, F.E5M2])
def test_quantiser_equals_brute_force_nearest(fmt):
    x = interesting_values(fmt, np.random.default_rng(1))
    got = F.quantise_codes(x, fmt)
    want = brute_force_nearest(x, fmt)
    bad = np.flatnonzero(got != want)
    assert bad.size == 0, (x[bad][:5], got[bad][:5], want[bad][:5])


@pytest.mark.parametrize("fmt", [F.E4M3, F.E5M2])
def test_quantiser_equals_library_cast_in_range(fmt):
    """torch's float32 -> float8 conversion rounds to nearest-even; compare wherever the
    result is finite (its overflow convention differs from the saturating cast)."""
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(1 << 20) * np.exp2(rng.integers(-22, 10 if fmt is F.E4M3 else 17, 1 << 20))).astype(np.float32)
    lib = torch.from_numpy(x).to(TORCH_FP8[fmt.name])
    libv = lib.to(torch.float64).numpy()
    libc = lib.view(torch.uint8).numpy()
    ok = np.isfinite(libv) & (np.abs(x) <= fmt.max_finite)
    assert ok.mean() > 0.9
    assert np.array_equal(F.quantise_codes(x, fmt)[ok], libc[ok])


@pytest.mark.parametrize("fmt", [F.E4M3, F.E5M2])
def test_saturation_and_specials(fmt):
    x = np.array([np.inf, -np.inf, 1e38, -1e38, fmt.max_finite * (1 + 2.0 ** -(fmt.M + 1)), np.nan])
    q = F.quantise(x, fmt)
    assert np.array_equal(q[:5], [fmt.max_finite, -fmt.max_finite, fmt.max_finite, -fmt.max_finite, fmt.max_finite])
    assert np.isnan(q[5]) and np.isnan(F.decode(F.quantise_codes(x, fmt), fmt)[5])
    z = F.quantise_codes(np.array([0.0, -0.0, fmt.min_subnormal * 0.5, -fmt.min_subnormal * 0.5]), fmt)
    assert list(z) == [0, 0x80, 0, 0x80]        # the exact half-way point ties to the even code 0


@pytest.mark.parametrize("fmt", [F.E4M3, F.E5M2])
def test_round_trip_idempotent_monotone_odd(fmt):
    codes = np.arange(256)
    vals = F.decode(codes, fmt)
    fin = np.isfinite(vals)
    assert np.array_equal(F.encode(vals[fin], fmt), codes[fin].astype(np.uint8))
    assert np.array_equal(F.quantise_codes(vals[fin], fmt), codes[fin].astype(np.uint8))
    x = np.sort(np.random.default_rng(3).standard_normal(100000) * 50)
    q = F.quantise(x, fmt)
    assert np.all(np.diff(q) >= 0)
    assert np.array_equal(F.quantise(-x, fmt), -q)
    assert np.array_equal(F.quantise(q, fmt), q)


def structured_fp32_patterns():
    """Every (sign, exponent, top-7-mantissa) prefix of float32 x 256 pseudo-random low halves: 2^24 patterns."""
    hi = np.arange(1 << 16, dtype=np.uint32)
    lo = np.random.default_rng(4).integers(0, 1 << 16, size=256, dtype=np.uint32)
    lo[:4] = [0, 1, 0x8000, 0xFFFF]
    bits = (hi[:, None] << 16 | lo[None, :]).reshape(-1)
    return bits.view(np.float32)


def test_fp16_equals_numpy_cast_on_structured_patterns():
    x = structured_fp32_patterns()
    with np.errstate(over="ignore", invalid="ignore"):
        lib = x.astype(np.float16)
    ours = F.quantise_codes(x, F.FP16)
    nan = np.isnan(x)
    assert np.array_equal(ours[~nan], lib.view(np.uint16)[~nan])
    assert np.all(np.isnan(F.decode(ours[nan], F.FP16)))


def test_bf16_equals_torch_cast_on_structured_patterns():
    x = structured_fp32_patterns()
    lib = torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    ours = F.quantise_codes(x, F.BF16)
    nan = np.isnan(x)
    assert np.array_equal(ours[~nan], lib[~nan])


def test_all_16bit_sources_decode_like_library():
    codes = np.arange(1 << 16, dtype=np.uint16)
    h = codes.view(np.float16).astype(np.float64)
    ours = F.decode(codes, F.FP16)
    ok = ~np.isnan(h)
    assert np.array_equal(ours[ok], h[ok]) and np.all(np.isnan(ours[~ok]))
    b = torch.from_numpy(codes.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    ours = F.decode(codes, F.BF16)
    ok = ~np.isnan(b)
    assert np.array_equal(ours[ok], b[ok]) and np.all(np.isnan(ours[~ok]))


def test_snr_one_mantissa_bit_is_a_factor_of_four():
    """Rounding noise power scales with spacing^2: one fewer mantissa bit => ~4x lower SNR;
    both formats are clipping-free for unit-normal data (section "Quantisation error")."""
    x = np.random.default_rng(5).standard_normal(2_000_000)
    s4, s5 = F.snr(x, F.E4M3), F.snr(x, F.E5M2)
    assert 3.6 < s4 / s5 < 4.4
    # Uniform rounding noise spacing^2/12 with spacing 2^(e-M) against a signal whose squared
    # mantissa averages between 1 and 4: SNR lies between 12 * 4^M and 48 * 4^M.
    for s, M in ((s4, 3), (s5, 2)):
        assert 12 * 4.0 ** M < s < 48 * 4.0 ** M


def test_scaled_cast_multiplies_in_float32():
    x = np.array([3.0000002, 1e-3, 123.456], dtype=np.float32)
    s = np.float32(0.1)
    want = F.quantise_codes((x * s).astype(np.float64), F.E4M3)
    assert np.array_equal(F.scaled_cast(x, 0.1, F.E4M3), want)


def test_folded_normal_mass_pin():
    """The paper prints that about 90 % of a unit normal's mass lies in [2^-4, 2^1]: the oracle's exponent histogram of a
    large unit-normal sample must put that share into the bins of exponents -4 .. 0, and the closed form agrees."""
    rng = np.random.default_rng(1)
    n = 400000
    h = F.exponent_histogram(rng.standard_normal(n), -4, 5)
    assert abs(h[1:6].sum() / n - GOLD["folded_normal_mass"]) < 0.01
    from scipy import special
    mass = special.erf(2 / np.sqrt(2)) - special.erf(2.0 ** -4 / np.sqrt(2))
    assert abs(h[1:6].sum() / n - mass) < 3e-3


def test_exponent_histogram_bins_by_floor_log2():
    x = np.array([0.0, -0.0, 1.0, -1.0, 1.5, 2.0, 3.999, 4.0, 0.5, 0.49, 2.0 ** -10, 2.0 ** 10, np.inf, np.nan, -7.0])
    h = F.exponent_histogram(x, -2, 5)          # bins for exponents -2 .. 2
    assert h.sum() == x.size
    #        below(<2^-2)  e=-2  e=-1  e=0  e=1  e=2  above
    assert h.tolist() == [3, 1, 1, 3, 2, 2, 3]      # 0.49 is in [2^-2, 2^-1), 0.5 in [2^-1, 1)
    # brute force with math.log2 on a random sample
    rng = np.random.default_rng(0)
    y = rng.standard_normal(5000) * 3
    ref = np.zeros(12, dtype=np.int64)
    import math
    for v in y:
        e = math.floor(math.log2(abs(v)))
        ref[0 if e < -6 else 11 if e >= 4 else 1 + e + 6] += 1
    assert np.array_equal(F.exponent_histogram(y, -6, 10), ref)
    # a unit-normal tensor has most of its mass in the exponents -3 .. 1 (figure of the appendix: narrow histogram)
    assert F.exponent_histogram(rng.standard_normal(100000), -3, 5)[1:6].sum() > 0.9 * 100000

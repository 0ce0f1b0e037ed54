"""Pins for the oracle's floating-point quantiser (Sec. 2.2 of the paper; SxEyMz notation, Sec. 3.1).

The oracle is checked against things other than itself: library casts at the two formats the
paper names by their IEEE names (S1E8M23 = FP32, S1E5M10 = FP16) and at bfloat16, a brute-force
nearest-value search in exact rational arithmetic, and the properties rounding to nearest must
have (half-spacing error bound, monotone, idempotent, odd).
"""
import bisect
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import omc_oracle as orc

# formats of the paper (Tables 1-2, Sec. 3.4, Sec. 3.5.3) and of the benchmark configurations
PAPER_FORMATS = [(4, 14), (3, 7), (2, 3), (5, 10), (3, 9), (4, 8), (5, 7), (8, 23)]
CONFIG_FORMATS = [(5, 2), (4, 3), (5, 6), (5, 10)]
SMALL_FORMATS = [(5, 2), (4, 3), (5, 6), (3, 7), (2, 3), (2, 0), (3, 0), (2, 1)]  # B <= 12


def bits(x):
    return np.asarray(x, np.float32).view(np.uint32)


def from_bits(u):
    return np.asarray(u, np.uint32).view(np.float32)


def sample_floats(rng, n, lo_exp=-40, hi_exp=20):
    """Random fp32 values spread over many binades, both signs."""
    mant = rng.uniform(1.0, 2.0, n)
    ex = rng.integers(lo_exp, hi_exp, n)
    sg = rng.choice([-1.0, 1.0], n)
    return (sg * mant * np.exp2(ex)).astype(np.float32)


def finite_values(E, M):
    """All non-negative finite values of SxEyMz from the IEEE parametrisation, as exact Fractions,
    with their magnitude codes, ascending."""
    bias = (1 << (E - 1)) - 1
    emin = 1 - bias
    vals = []
    for f in range(0, (1 << E) - 1):
        for m in range(1 << M):
            if f == 0:
                v = Fraction(m) * Fraction(2) ** (emin - M)
            else:
                v = (1 + Fraction(m, 1 << M)) * Fraction(2) ** (f - bias)
            vals.append((v, (f << M) | m))
    return vals


# ---------------------------------------------------------------------------------------------
# library casts

def test_s1e8m23_is_fp32_identity():
    rng = np.random.default_rng(0)
    u = rng.integers(0, 2 ** 32, 200000, dtype=np.uint64).astype(np.uint32)
    u = np.concatenate([u, np.array([0, 0x80000000, 1, 0x80000001, 0x7F800000, 0xFF800000,
                                     0x7FC00000, 0xFFC00001, 0x7F800001, 0x007FFFFF, 0x00800000,
                                     0x7F7FFFFF], np.uint32)])
    assert np.array_equal(orc.encode(from_bits(u), 8, 23), u)
    assert np.array_equal(bits(orc.decode(u, 8, 23)), u)


def test_s1e5m10_is_ieee_half_encode():
    rng = np.random.default_rng(1)
    x = np.concatenate([
        sample_floats(rng, 200000, -30, 18),
        rng.standard_normal(100000).astype(np.float32) * np.float32(0.05),
        np.array([0.0, -0.0, 65504.0, 65519.996, 65520.0, 65536.0, 1e30, -1e30, np.inf, -np.inf,
                  2.0 ** -24, 2.0 ** -25, np.nextafter(np.float32(2.0 ** -25), np.float32(1)),
                  2.0 ** -14, np.nextafter(np.float32(2.0 ** -14), np.float32(0)), 1e-45, -1e-45,
                  1.0009765625, 1.00048828125, 1.00146484375], np.float32)])
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16).astype(np.uint32)
    assert np.array_equal(orc.encode(x, 5, 10), want)
    # quiet NaNs whose payload survives in the top 10 bits agree with the library too
    nan = from_bits(np.array([0x7FC00000, 0xFFC00000, 0x7FE00000, 0x7FFFE000], np.uint32))
    assert np.array_equal(orc.encode(nan, 5, 10), nan.astype(np.float16).view(np.uint16))


def test_s1e5m10_is_ieee_half_decode_all_codes():
    codes = np.arange(65536, dtype=np.uint32)
    want = codes.astype(np.uint16).view(np.float16).astype(np.float32)
    assert np.array_equal(bits(orc.decode(codes, 5, 10)), bits(want))


def test_s1e8m7_is_bfloat16():
    rng = np.random.default_rng(2)
    x = np.concatenate([sample_floats(rng, 200000, -140, 127),
                        from_bits(rng.integers(0, 0x00800000, 1000).astype(np.uint32)),  # subnormal
                        np.array([0.0, -0.0, np.inf, -np.inf, 3.3895314e38, 3.4e38], np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.encode(x, 8, 7), want.astype(np.uint32))
    codes = np.arange(65536, dtype=np.uint32)
    back = torch.from_numpy(codes.astype(np.uint16).view(np.int16)).view(torch.bfloat16).float()
    assert np.array_equal(bits(orc.decode(codes, 8, 7)), bits(back.numpy()))


# ---------------------------------------------------------------------------------------------
# every code of the small formats and of FP16 survives decode -> encode

@pytest.mark.parametrize("E,M", SMALL_FORMATS + [(5, 10)])
def test_exhaustive_decode_encode_identity(E, M):
    B = 1 + E + M
    codes = np.arange(1 << B, dtype=np.uint32)
    vals = orc.decode(codes, E, M)
    back = orc.encode(vals, E, M)
    assert np.array_equal(back, codes)           # NaN payloads included (none exist when M = 0)
    # finite codes decode to distinct values except +0 / -0
    finite = np.isfinite(vals)
    assert np.unique(vals[finite]).size == finite.sum() - 1


@pytest.mark.parametrize("E,M", SMALL_FORMATS)
def test_decode_matches_ieee_parametrisation(E, M):
    for v, mag in finite_values(E, M):
        got = orc.decode(np.array([mag, mag | (1 << (E + M))], np.uint32), E, M)
        assert Fraction(float(got[0])) == v and Fraction(float(got[1])) == -v
    inf = ((1 << E) - 1) << M
    assert orc.decode([inf], E, M)[0] == np.inf and orc.decode([inf | 1 << (E + M)], E, M)[0] == -np.inf
    if M:
        assert np.isnan(orc.decode([inf | 1], E, M)[0])


# ---------------------------------------------------------------------------------------------
# rounding to nearest, ties to even: brute force in exact arithmetic

def brute_force_code(x, vals, E, M):
    """Nearest finite value by exact comparison; ties to even mantissa; IEEE overflow rule."""
    a = abs(Fraction(float(x)))
    sign = (1 << (E + M)) if np.signbit(x) else 0
    inf = ((1 << E) - 1) << M
    vmax = vals[-1][0]
    emax = (1 << (E - 1)) - 1
    if a >= vmax + (Fraction(2) ** (emax - M)) / 2:   # half a spacing above the largest value
        return sign | inf
    best, best_code = None, None
    for v, code in vals:
        d = abs(v - a)
        if best is None or d < best or (d == best and code % 2 == 0 and best_code % 2 == 1):
            best, best_code = d, code
    return sign | best_code


@pytest.mark.parametrize("E,M", [(2, 3), (4, 3), (5, 2), (3, 7), (2, 0), (2, 1)])
def test_round_to_nearest_even_brute_force_full_scan(E, M):
    rng = np.random.default_rng(10 + E * 31 + M)
    vals = finite_values(E, M)
    bias = (1 << (E - 1)) - 1
    xs = list(sample_floats(rng, 300, 1 - bias - M - 3, bias + 3))
    # adversarial: exact midpoints, just off midpoints, representable values, zero, tiny
    fl = [float(v) for v, _ in vals]
    for i in rng.choice(len(fl) - 1, 60):
        mid = np.float32((fl[i] + fl[i + 1]) / 2)          # exact in fp32 (M + 1 <= 24 bits)
        xs += [mid, np.nextafter(mid, np.float32(np.inf)), np.nextafter(mid, np.float32(0)),
               np.float32(fl[i]), -mid]
    top = np.float32(fl[-1])
    half = np.float32(2.0 ** (bias - M - 1))
    xs += [top, top + half, np.nextafter(top + half, np.float32(0)), np.float32(2.0 ** (bias + 1)),
           np.float32(0.0), np.float32(-0.0), np.float32(1e-45), np.float32(fl[1] / 2),
           np.nextafter(np.float32(fl[1] / 2), np.float32(1)), np.float32(fl[1] / 4)]
    xs = np.array(xs, np.float32)
    got = orc.encode(xs, E, M)
    for x, g in zip(xs, got):
        assert int(g) == brute_force_code(x, vals, E, M), (float(x), hex(int(g)))


@pytest.mark.parametrize("E,M", [(5, 6), (4, 8), (3, 9), (5, 7), (4, 14), (5, 10)])
def test_round_to_nearest_even_bracketing(E, M):
    """Larger formats: compare with the nearer of the two bracketing values (exact fractions)."""
    rng = np.random.default_rng(100 + E * 31 + M)
    bias = (1 << (E - 1)) - 1
    vals = finite_values(E, M)
    keys = [v for v, _ in vals]
    xs = sample_floats(rng, 4000, 1 - bias - M - 2, bias + 1)
    mids = []
    for i in rng.choice(len(keys) - 1, 400):
        mid = np.float32(float((keys[i] + keys[i + 1]) / 2))
        mids += [mid, -mid, np.nextafter(mid, np.float32(np.inf)), np.nextafter(mid, np.float32(0))]
    xs = np.concatenate([xs, np.array(mids, np.float32)])
    got = orc.encode(xs, E, M)
    sign_bit = 1 << (E + M)
    inf = ((1 << E) - 1) << M
    for x, g in zip(xs, got):
        a = abs(Fraction(float(x)))
        g = int(g)
        assert (g & sign_bit != 0) == bool(np.signbit(x))
        g &= sign_bit - 1
        hi = bisect.bisect_left(keys, a)
        if hi == len(keys):
            over = a >= keys[-1] + (Fraction(2) ** (bias - M)) / 2
            assert g == (inf if over else vals[-1][1])
            continue
        if keys[hi] == a:
            assert g == vals[hi][1]
            continue
        lo = hi - 1
        dlo, dhi = a - keys[lo], keys[hi] - a
        if dlo < dhi:
            want = vals[lo][1]
        elif dhi < dlo:
            want = vals[hi][1]
        else:
            want = vals[lo][1] if vals[lo][1] % 2 == 0 else vals[hi][1]
        assert g == want, (float(x), hex(g), hex(want))


@pytest.mark.parametrize("E,M", sorted(set(PAPER_FORMATS + CONFIG_FORMATS + [(8, 7), (2, 0), (7, 22),
                                                                             (4, 23)])))
def test_rounding_properties(E, M):
    rng = np.random.default_rng(1000 + E * 31 + M)
    bias = (1 << (E - 1)) - 1
    emin, emax = 1 - bias, bias
    lo = max(emin - M - 3, -148)
    x = np.sort(sample_floats(rng, 20000, lo, min(emax + 2, 127)))
    c = orc.encode(x, E, M)
    q = orc.decode(c, E, M)
    # (ii) half-spacing error bound for in-range values
    inr = np.abs(x.astype(np.float64)) < 2.0 ** emax * (2 - 2.0 ** -(M + 1))
    e = np.floor(np.log2(np.abs(x[inr].astype(np.float64))))
    half = np.exp2(np.maximum(e, emin) - M - 1)
    err = np.abs(q[inr].astype(np.float64) - x[inr].astype(np.float64))
    assert np.all(err <= half)
    assert np.all(np.isinf(q[~inr]))
    # (iii) monotone (x is sorted)
    assert not np.isnan(q).any()
    qi = np.clip(q.astype(np.float64), -1e300, 1e300)          # infinities ordered at the ends
    assert np.all(np.diff(qi) >= 0)
    # (iv) idempotent, (v) odd
    assert np.array_equal(orc.encode(q, E, M), c)
    assert np.array_equal(orc.encode(-x, E, M), c ^ np.uint32(1 << (E + M)))


@pytest.mark.parametrize("E,M", [(5, 2), (4, 3), (5, 6), (3, 7), (4, 14), (5, 10)])
def test_boundaries(E, M):
    bias = (1 << (E - 1)) - 1
    emin, emax = 1 - bias, bias
    inf = ((1 << E) - 1) << M
    top = np.float32(2.0 ** emax * (2 - 2.0 ** -M))
    thr = np.float32(2.0 ** emax * (2 - 2.0 ** -(M + 1)))     # tie between top and 2^(emax+1)
    assert orc.encode([top], E, M)[0] == inf - 1
    assert orc.encode([thr], E, M)[0] == inf                  # ties to even -> overflow
    assert orc.encode([np.nextafter(thr, np.float32(0))], E, M)[0] == inf - 1
    tiny = 2.0 ** (emin - M)                                  # smallest subnormal
    assert orc.encode([np.float32(tiny)], E, M)[0] == 1
    assert orc.encode([np.float32(tiny / 2)], E, M)[0] == 0   # tie -> even (zero)
    assert orc.encode([np.nextafter(np.float32(tiny / 2), np.float32(1))], E, M)[0] == 1
    assert orc.encode([np.float32(1.5 * tiny)], E, M)[0] == 2  # tie -> even
    assert orc.encode([np.float32(-tiny / 2)], E, M)[0] == 1 << (E + M)   # -0 keeps its sign
    # largest subnormal rounds up into the first normal binade
    edge = np.nextafter(np.float32(2.0 ** emin), np.float32(0))
    assert orc.encode([edge], E, M)[0] == 1 << M
    # carry out of the mantissa into the exponent
    x = np.nextafter(np.float32(2.0), np.float32(0))
    if M < 23 and emax >= 1:
        assert orc.decode(orc.encode([x], E, M), E, M)[0] == 2.0


def test_nan_reading():
    # payload only in low bits: a quiet bit is forced (reading; the library cast differs here)
    x = from_bits(np.array([0x7F800001, 0xFF800001], np.uint32))
    assert list(orc.encode(x, 5, 10)) == [0x7E00, 0xFE00]
    assert list(orc.encode(x, 5, 2)) == [0x7E, 0xFE]
    # M = 0 has no NaN code: infinity of that sign
    assert list(orc.encode(x, 2, 0)) == [0b011, 0b111]

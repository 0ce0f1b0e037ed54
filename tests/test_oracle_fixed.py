"""Pins for the oracle's fixed-point codec variant (Sec. 2.2 mentions fixed-point formats without
defining one: S1IxFy, two's complement, value k * 2^-y, round to nearest even, saturating, is this
library's reading).  What the mathematics fixes: decode -> encode is the identity on every code,
encode returns the nearest representable value (brute force in exact rationals), the error is at
most half a step inside the range, encode is monotone and idempotent, and Q15 / Q7 equal numpy's
round-and-clip to int16 / int8."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import omc_oracle as orc

FORMATS = [(0, 7), (0, 11), (0, 15), (1, 6), (2, 3), (3, 0), (0, 1), (4, 11), (8, 15), (0, 23)]


def values_of(I, F):
    B = 1 + I + F
    return [Fraction(k, 2 ** F) for k in range(-2 ** (B - 1), 2 ** (B - 1))]


@pytest.mark.parametrize("I,F", [f for f in FORMATS if 1 + f[0] + f[1] <= 16], ids=lambda v: str(v))
def test_every_code_decodes_and_encodes_back(I, F):
    B = 1 + I + F
    codes = np.arange(2 ** B, dtype=np.uint32)
    vals = orc.decode(codes, I, F, fixed=True)
    assert np.array_equal(orc.encode(vals, I, F, fixed=True), codes)
    # two's complement, value k 2^-F: exact, ordered like the signed integers
    k = np.where(codes >= 2 ** (B - 1), codes.astype(np.int64) - 2 ** B, codes.astype(np.int64))
    assert np.array_equal(vals.astype(np.float64), k / 2.0 ** F)
    assert vals[2 ** B - 1] == -(2.0 ** -F) and vals[2 ** (B - 1)] == -(2.0 ** I) and vals[0] == 0.0


@pytest.mark.parametrize("I,F", [(0, 3), (1, 2), (2, 3), (0, 7), (3, 0)], ids=lambda v: str(v))
def test_encode_is_the_nearest_value_ties_to_even(I, F):
    """Brute force over all representable values in exact rationals."""
    vals = values_of(I, F)
    B = 1 + I + F
    rng = np.random.default_rng(I * 10 + F)
    xs = list((rng.standard_normal(1500) * 2.0 ** I).astype(np.float32))
    step = 2.0 ** -F
    xs += [np.float32(v) for k in range(-2 ** (B - 1) - 2, 2 ** (B - 1) + 2) for v in
           ((k + 0.5) * step, np.nextafter(np.float32((k + 0.5) * step), np.float32(9)),
            np.nextafter(np.float32((k + 0.5) * step), np.float32(-9)))]          # every tie and its neighbours
    xs += [np.float32(v) for v in (0.0, -0.0, 1e-30, -1e-30, 1e30, -1e30, 3.4e38, -3.4e38, 1e-45)]
    got = orc.decode(orc.encode(xs, I, F, fixed=True), I, F, fixed=True)
    for x, g in zip(xs, got):
        fx = Fraction(float(x))
        best = min(abs(v - fx) for v in vals)
        cands = [v for v in vals if abs(v - fx) == best]
        if len(cands) == 2:                              # an exact tie: the even multiple of the step
            cands = [v for v in cands if (v * 2 ** F) % 2 == 0]
        assert Fraction(float(g)) == cands[0], (x, g, cands)


@pytest.mark.parametrize("I,F", FORMATS, ids=lambda v: str(v))
def test_half_step_bound_saturation_monotone_idempotent(I, F):
    rng = np.random.default_rng(F + 100 * I)
    lo, hi = -2.0 ** I, 2.0 ** I - 2.0 ** -F
    x = np.sort((rng.uniform(-1.5, 1.5, 20000) * 2.0 ** I).astype(np.float32))
    q = orc.decode(orc.encode(x, I, F, fixed=True), I, F, fixed=True).astype(np.float64)
    inside = (x >= lo) & (x <= hi)
    assert np.all(np.abs(q[inside] - x[inside].astype(np.float64)) <= 2.0 ** -(F + 1))
    assert np.all(q[x > hi] == hi) and np.all(q[x < lo] == lo)          # saturation, no infinity
    assert np.all(np.diff(q) >= 0)                                     # monotone
    assert np.array_equal(orc.encode(q.astype(np.float32), I, F, fixed=True), orc.encode(x, I, F, fixed=True))
    sp = orc.decode(orc.encode([np.inf, -np.inf, np.nan], I, F, fixed=True), I, F, fixed=True)
    assert sp[0] == hi and sp[1] == lo and sp[2] == 0.0


@pytest.mark.parametrize("F,dtype", [(15, np.int16), (7, np.int8)])
def test_q15_and_q7_equal_numpy_round_and_clip(F, dtype):
    rng = np.random.default_rng(F)
    x = np.concatenate([(rng.standard_normal(50000) * 0.4).astype(np.float32),
                        (np.arange(-40, 40) + 0.5).astype(np.float32) * np.float32(2.0 ** -F),
                        np.array([1.0, -1.0, 0.99999, -1.00001, 2.0, -2.0], np.float32)])
    info = np.iinfo(dtype)
    want = np.clip(np.rint(x.astype(np.float64) * 2.0 ** F), info.min, info.max).astype(dtype)   # rint: ties to even
    got = orc.encode(x, 0, F, fixed=True)
    assert np.array_equal(got.astype(np.uint16 if F == 15 else np.uint8).view(dtype), want)


def test_fixed_point_variable_round_trip_and_update():
    """The whole-variable operations with the fixed-point codec: codes are encode(V) packed, the fit
    is the same least squares (pinned elsewhere) on (V, decode(encode(V))), the update path is
    decompress -> fma -> compress in exact rationals."""
    from test_oracle_pack_fit import f32_round, exact_least_squares
    I, F = 0, 7
    rng = np.random.default_rng(1)
    V = (rng.standard_normal(400) * 0.3).astype(np.float32)
    packed, s, b = orc.compress_var(V, I, F, fixed=True)
    codes = orc.encode(V, I, F, fixed=True)
    assert np.array_equal(orc.unpack(packed, V.size, 8), codes)
    Vt = orc.decode(codes, I, F, fixed=True)
    s_ex, b_ex = exact_least_squares(V, Vt)
    assert s == f32_round(s_ex) and b == f32_round(b_ex)
    assert np.linalg.norm(orc.decompress_var(packed, V.size, I, F, s, b, fixed=True) - V) <= np.linalg.norm(Vt - V) * (1 + 1e-6)
    g = (rng.standard_normal(400) * 0.1).astype(np.float32)
    new_packed, s2, b2, W = orc.update_recompress_var(packed, V.size, I, F, s, b, g, 0.5, want_w=True, fixed=True)
    lr = Fraction(0.5)
    for k in range(0, 400, 7):
        vbar = f32_round(Fraction(float(s)) * Fraction(float(Vt[k])) + Fraction(float(b)))
        w = f32_round(Fraction(float(vbar)) - lr * Fraction(float(g[k])))
        assert W[k] == w
    assert np.array_equal(orc.unpack(new_packed, V.size, 8), orc.encode(W, I, F, fixed=True))


def test_fixed_format_limits():
    L = orc.lib()
    assert L.orc_fixed_format_ok(0, 7) and L.orc_fixed_format_ok(8, 15) and L.orc_fixed_format_ok(0, 23)
    assert not L.orc_fixed_format_ok(0, 0) and not L.orc_fixed_format_ok(1, 23) and not L.orc_fixed_format_ok(9, 3)

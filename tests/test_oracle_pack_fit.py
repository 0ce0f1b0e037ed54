"""Pins for the oracle's bit packing, exact summation, per-variable transformation fit (Sec. 2.3)
and the update path (Sec. 2.1)."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import omc_oracle as orc


def f32_round(fr: Fraction) -> np.float32:
    """Correctly rounded fp32 (nearest, ties to even) of an exact rational, by comparing the exact
    distances to the neighbouring fp32 values."""
    c = np.float32(float(fr))
    cands = {c, np.nextafter(c, np.float32(np.inf)), np.nextafter(c, np.float32(-np.inf))}
    best = None
    for v in cands:
        if not np.isfinite(v):
            continue
        d = abs(Fraction(float(v)) - fr)
        even = (int(np.float32(v).view(np.uint32)) & 1) == 0
        if best is None or d < best[0] or (d == best[0] and even):
            best = (d, v)
    return np.float32(best[1])


# ---------------------------------------------------------------------------------------------
# packing

def test_pack_hand_examples():
    # B = 3: codes 1..7,0 -> bit stream written out by hand (least significant bit first)
    got = orc.pack([1, 2, 3, 4, 5, 6, 7, 0], 3)
    assert got.size == 16 and list(got[:3]) == [0xD1, 0x58, 0x1F] and not got[3:].any()
    got = orc.pack([0xABC, 0x123], 12)
    assert list(got[:3]) == [0xBC, 0x3A, 0x12] and not got[3:].any()
    got = orc.pack([0x1234, 0xBEEF], 16)
    assert list(got[:4]) == [0x34, 0x12, 0xEF, 0xBE]
    got = orc.pack([0x5A], 8)
    assert got[0] == 0x5A and got.size == 16
    got = orc.pack([0x12345, 0x7FFFF], 19)        # 38 bits
    v = 0x12345 | (0x7FFFF << 19)
    assert list(got[:5]) == [(v >> (8 * i)) & 0xFF for i in range(5)]


@pytest.mark.parametrize("B", [3, 6, 8, 11, 12, 13, 16, 19, 24, 32])
def test_pack_unpack_identity_and_padding(B):
    rng = np.random.default_rng(B)
    for n in [1, 2, 7, 127, 128, 129, 1000]:
        codes = rng.integers(0, 2 ** B, n, dtype=np.uint64).astype(np.uint32)
        p = orc.pack(codes, B)
        assert p.size % 16 == 0 and p.size == (((n * B + 7) // 8 + 15) // 16) * 16
        assert np.array_equal(orc.unpack(p, n, B), codes)
        stream = np.unpackbits(p, bitorder="little")
        assert not stream[n * B:].any()                       # zero padding
        want = ((codes[:, None] >> np.arange(B, dtype=np.uint32)) & 1).astype(np.uint8).ravel()
        assert np.array_equal(stream[:n * B], want)


# ---------------------------------------------------------------------------------------------
# exact summation against the library's correctly rounded sum

def test_exact_sum_matches_fsum():
    rng = np.random.default_rng(5)
    cases = [
        rng.standard_normal(5000) * np.exp(rng.uniform(-40, 40, 5000)),
        np.array([1e300, 1.0, -1e300, 1e-300, 3.0]),
        np.array([2.0 ** 53, 1.0, 1.0, -2.0 ** 53]),
        np.array([2.0 ** 53, 1.0]),                       # tie -> even
        np.array([2.0 ** 53, 3.0]),                       # tie -> even, other way
        np.array([2.0 ** 53, 1.0, 2.0 ** -60]),           # sticky bit breaks the tie
        np.array([5e-324, 5e-324, -5e-324, 2.5e-320]),
        -np.abs(rng.standard_normal(1000)) * 1e-20,
        (rng.standard_normal(3000).astype(np.float32).astype(np.float64)) ** 2,
        np.zeros(10),
    ]
    for x in cases:
        assert orc.exact_sum(x) == math.fsum(x), x[:5]
    assert orc.exact_sum(np.array([1.7e308, 1.7e308])) == np.inf
    assert orc.exact_sum(np.array([1.7e308, 1.7e308, -1.7e308])) == 1.7e308   # no intermediate overflow
    assert orc.exact_sum(np.array([np.inf, 1.0])) == np.inf
    assert math.isnan(orc.exact_sum(np.array([np.inf, -np.inf])))


# ---------------------------------------------------------------------------------------------
# per-variable transformation

def exact_least_squares(V, Vt):
    """Solve min ||s*Vt + b - V||_2 exactly: normal equations by elimination over the rationals."""
    x = [Fraction(float(t)) for t in Vt]
    y = [Fraction(float(v)) for v in V]
    n = len(x)
    a11, a12, a22 = sum(t * t for t in x), sum(x), Fraction(n)
    r1, r2 = sum(t * v for t, v in zip(x, y)), sum(y)
    # [a11 a12; a12 a22] [s; b] = [r1; r2]
    f = a12 / a11
    b = (r2 - f * r1) / (a22 - f * a12)
    s = (r1 - a12 * b) / a11
    return s, b


@pytest.mark.parametrize("E,M,scale,mean", [(5, 2, 0.05, 0.0), (4, 3, 0.1, 0.02), (5, 6, 0.02, 0.0),
                                            (3, 7, 0.3, -0.1), (5, 10, 0.05, 0.001), (2, 3, 1.0, 0.5)])
def test_fit_is_exact_least_squares(E, M, scale, mean):
    rng = np.random.default_rng(E * 100 + M)
    for n in [2, 3, 17, 500]:
        V = (rng.standard_normal(n) * scale + mean).astype(np.float32)
        Vt = orc.decode(orc.encode(V, E, M), E, M)
        if np.unique(Vt).size < 2:
            continue
        s, b, sums = orc.fit(V, Vt, want_sums=True)
        s_ex, b_ex = exact_least_squares(V, Vt)
        assert s == f32_round(s_ex) and b == f32_round(b_ex)
        # normal equations hold for the exact solution; the stored fp32 pair is its rounding
        r = [Fraction(float(v)) - s_ex * Fraction(float(t)) - b_ex for v, t in zip(V, Vt)]
        assert sum(r) == 0 and sum(ri * Fraction(float(t)) for ri, t in zip(r, Vt)) == 0
        # the four sums are the correctly rounded exact sums
        V64, T64 = V.astype(np.float64), Vt.astype(np.float64)
        assert list(sums) == [math.fsum(V64), math.fsum(T64), math.fsum(V64 * T64),
                              math.fsum(T64 * T64)]


def test_fit_matches_library_regression():
    rng = np.random.default_rng(77)
    V = (rng.standard_normal(4096) * 0.05 + 0.01).astype(np.float32)
    Vt = orc.decode(orc.encode(V, 5, 2), 5, 2)
    s, b = orc.fit(V, Vt)
    A = np.stack([Vt.astype(np.float64), np.ones(V.size)], 1)
    (s_l, b_l), *_ = np.linalg.lstsq(A, V.astype(np.float64), rcond=None)
    assert abs(s - s_l) <= 1e-6 * abs(s_l) and abs(b - b_l) <= 1e-6 * max(abs(b_l), 1e-3)
    p = np.polyfit(Vt.astype(np.float64), V.astype(np.float64), 1)
    assert abs(s - p[0]) <= 1e-6 * abs(p[0])


def test_fit_reduces_error_and_lossless_gives_identity():
    rng = np.random.default_rng(78)
    V = (rng.standard_normal(20000) * 0.05).astype(np.float32)
    for E, M in [(5, 2), (4, 3), (3, 7), (2, 3)]:
        Vt = orc.decode(orc.encode(V, E, M), E, M)
        s, b = orc.fit(V, Vt)
        e_plain = np.sum((V.astype(np.float64) - Vt) ** 2)
        e_pvt = np.sum((V.astype(np.float64) - (float(s) * Vt.astype(np.float64) + float(b))) ** 2)
        assert e_pvt <= e_plain
    s, b = orc.fit(V, V)                       # lossless code: Vt == V
    assert s == 1.0 and b == 0.0
    s, b = orc.fit(V, V, pvt=False)
    assert s == 1.0 and b == 0.0


def test_printed_closed_forms_do_not_solve_the_stated_minimisation():
    """Sec. 2.3 prints s with n*Sum(V^2) in the denominator and b with n*Sum(V) in the numerator.
    With a lossless code (Vt == V) the minimiser of the stated objective is s = 1, b = 0; the
    printed b does not give that, the normal-equation solution does (it is what the oracle uses)."""
    V = [Fraction(1), Fraction(2), Fraction(4)]
    n = len(V)
    Sx = sum(V); Sxx = sum(v * v for v in V)
    s_printed = (n * Sxx - Sx * Sx) / (n * Sxx - Sx * Sx)
    b_printed = (n * Sx - s_printed * Sx) / n
    assert s_printed == 1 and b_printed != 0
    s, b = exact_least_squares([float(v) for v in V], [float(v) for v in V])
    assert s == 1 and b == 0


def test_fit_affine_equivariance():
    rng = np.random.default_rng(79)
    V = (rng.standard_normal(3000) * 0.05).astype(np.float32)
    Vt = orc.decode(orc.encode(V, 5, 2), 5, 2)
    s, b = orc.fit(V, Vt)
    alpha, beta = 4.0, 0.25                                  # exact in fp32
    s2, b2 = orc.fit((alpha * V + beta).astype(np.float32), Vt)
    assert abs(s2 - alpha * s) <= 2e-6 * abs(alpha * s)
    assert abs(b2 - (alpha * b + beta)) <= 2e-6 * abs(alpha * b + beta)


def test_fit_degenerate_cases():
    # all elements equal (Sec. 2.3: denominator 0): s = 1, b makes the mean match
    V = np.full(100, 0.3, np.float32)
    Vt = orc.decode(orc.encode(V, 5, 2), 5, 2)
    s, b = orc.fit(V, Vt)
    assert s == 1.0 and b == np.float32(np.float64(V[0]) - np.float64(Vt[0]))
    # one element
    s, b = orc.fit(np.array([0.3], np.float32), np.array([0.25], np.float32))
    assert s == 1.0 and b == np.float32(np.float64(np.float32(0.3)) - 0.25)
    # all zero
    s, b = orc.fit(np.zeros(10, np.float32), np.zeros(10, np.float32))
    assert s == 1.0 and b == 0.0
    # all values inside one quantisation cell: Vt constant, V not
    V = np.linspace(0.26, 0.27, 1000).astype(np.float32)
    Vt = orc.decode(orc.encode(V, 5, 2), 5, 2)
    assert np.unique(Vt).size == 1
    s, b = orc.fit(V, Vt)
    mean_gap = (math.fsum(V.astype(np.float64)) - math.fsum(Vt.astype(np.float64))) / V.size
    assert s == 1.0 and b == np.float32(mean_gap)
    # a large constant whose fp64 denominator would not cancel exactly without the exact test
    V = np.full(100003, 1.1, np.float32)
    s, b = orc.fit(V, V)
    assert s == 1.0 and b == 0.0
    # mixed signed zeros are equal values
    Vt = np.array([0.0, -0.0, 0.0], np.float32)
    s, b = orc.fit(np.array([1e-9, -1e-9, 0], np.float32), Vt)
    assert s == 1.0


def test_fit_non_finite():
    V = np.array([1.0, np.inf, 2.0], np.float32)
    s, b = orc.fit(V, V)
    assert s == 1.0 and not np.isfinite(b)
    V = np.array([1.0, np.nan, 2.0], np.float32)
    s, b = orc.fit(V, V)
    assert s == 1.0 and np.isnan(b)


# ---------------------------------------------------------------------------------------------
# whole-variable operations

@pytest.mark.parametrize("E,M", [(5, 2), (4, 3), (5, 6), (5, 10), (3, 7), (4, 14)])
def test_compress_decompress_var(E, M):
    rng = np.random.default_rng(E * 7 + M)
    n = 1001
    V = (rng.standard_normal(n) * 0.05).astype(np.float32)
    packed, s, b = orc.compress_var(V, E, M)
    codes = orc.encode(V, E, M)
    assert np.array_equal(packed, orc.pack(codes, 1 + E + M))
    Vt = orc.decode(codes, E, M)
    assert (s, b) == orc.fit(V, Vt)
    out = orc.decompress_var(packed, n, E, M, s, b)
    want = np.array([f32_round(Fraction(float(s)) * Fraction(float(t)) + Fraction(float(b)))
                     for t in Vt], np.float32)
    assert np.array_equal(out.view(np.uint32), want.view(np.uint32))
    # inverse-transform consistency: the transformed reconstruction is at least as close
    err_t = np.linalg.norm(V.astype(np.float64) - out)
    err_p = np.linalg.norm(V.astype(np.float64) - Vt)
    assert err_t <= err_p * (1 + 1e-6)


@pytest.mark.parametrize("lr", [0.01, 10.0])
def test_update_recompress_var(lr):
    """W = fl32(Vbar - lr*g) with Vbar = fl32(s*Vt + b), each one rounding, then compression of W.
    lr = 10 makes the step larger than the code spacing so that codes really change."""
    E, M, n = 5, 2, 777
    rng = np.random.default_rng(3)
    V = (rng.standard_normal(n) * 0.05).astype(np.float32)
    g = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    packed, s, b = orc.compress_var(V, E, M)
    new_packed, s2, b2, W = orc.update_recompress_var(packed, n, E, M, s, b, g, lr, want_w=True)
    Vt = orc.decode(orc.unpack(packed, n, 1 + E + M), E, M)
    lr32 = Fraction(float(np.float32(lr)))
    for k in range(n):
        vbar = f32_round(Fraction(float(s)) * Fraction(float(Vt[k])) + Fraction(float(b)))
        w = f32_round(Fraction(float(vbar)) - lr32 * Fraction(float(g[k])))
        assert W[k].view(np.uint32) == w.view(np.uint32)
    p3, s3, b3 = orc.compress_var(W, E, M)
    assert np.array_equal(new_packed, p3) and (s2, b2) == (s3, b3)
    changed = np.count_nonzero(orc.unpack(new_packed, n, 8) != orc.unpack(packed, n, 8))
    assert (changed > n // 10) if lr == 10.0 else True
    # FP32 variables: plain SGD with one rounding
    v2 = orc.sgd_var(V, g, lr)
    for k in range(0, n, 50):
        assert v2[k] == f32_round(Fraction(float(V[k])) - lr32 * Fraction(float(g[k])))


def test_update_nan_is_canonical():
    E, M = 5, 2
    V = np.array([0.1, np.inf, 0.2, -0.3], np.float32)
    packed, s, b = orc.compress_var(V, E, M)
    assert s == 1.0 and not np.isfinite(b)
    g = np.zeros(4, np.float32)
    new_packed, s2, b2, W = orc.update_recompress_var(packed, 4, E, M, s, b, g, 0.01, want_w=True)
    nanmask = np.isnan(W)
    assert nanmask.any()
    assert np.all(W.view(np.uint32)[nanmask] == 0x7FFFFFFF)
    codes = orc.unpack(new_packed, 4, 8)
    assert np.all(codes[nanmask] == 0x7F)


# ---------------------------------------------------------------------------------------------
# server-side mean of the clients' models (Sec. 1, Sec. 2.5)

@pytest.mark.parametrize("K", [1, 2, 3, 5, 8, 16])
def test_aggregate_var_is_the_sequentially_rounded_mean(K):
    """FP32 additions in client order, one rounded division: every step in exact rationals."""
    rng = np.random.default_rng(K)
    n = 60
    xs = [(rng.standard_normal(n) * 10.0 ** rng.integers(-3, 3)).astype(np.float32) for _ in range(K)]
    xs[0][:4] = [1e30, 1.0, -0.0, 3.0]
    if K >= 3:
        xs[1][:4] = [1.0, 1e-8, 0.0, 1e-45]
        xs[2][:4] = [-1e30, -1.0, -0.0, 2e-45]      # order matters: (1e30 + 1) - 1e30 = 0, not 1
    got = orc.aggregate_var(xs)
    for e in range(n):
        acc = np.float32(xs[0][e])
        for k in range(1, K):
            acc = f32_round(Fraction(float(acc)) + Fraction(float(xs[k][e])))
        want = f32_round(Fraction(float(acc)) / K)
        assert got[e] == want, (e, got[e], want)
    if K >= 3:
        assert got[0] == 0.0 or K > 3                 # the cancellation case above, clients in order
    if K == 1:
        assert np.array_equal(got.view(np.uint32), xs[0].view(np.uint32))


def test_aggregate_var_invariants():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(500)).astype(np.float32)
    # identical clients: x + x and its half are exact; with few significant bits every partial
    # sum k x is exact too, and so is the division for any K
    assert np.array_equal(orc.aggregate_var([x, x]), x)
    coarse = np.round(x * 1024).astype(np.float32) / np.float32(1024)
    for K in (3, 4, 7, 16):
        assert np.array_equal(orc.aggregate_var([coarse] * K), coarse)
    # the mean lies between the smallest and the largest client value
    xs = [(x + rng.standard_normal(500).astype(np.float32) * np.float32(0.1)) for _ in range(7)]
    m = orc.aggregate_var(xs)
    lo, hi = np.min(xs, axis=0), np.max(xs, axis=0)
    tol = 7 * 2.0 ** -23 * np.max(np.abs(xs), axis=0)        # six additions and a division, each within half an ulp
    assert np.all(m >= lo - tol) and np.all(m <= hi + tol)
    # non-finite values follow IEEE-754: Inf + (-Inf) = NaN, Inf stays Inf
    a = np.array([np.inf, np.inf, 1.0], np.float32)
    b = np.array([-np.inf, 1.0, np.nan], np.float32)
    got = orc.aggregate_var([a, b])
    assert np.isnan(got[0]) and got[1] == np.inf and np.isnan(got[2])


def test_aggregate_models_decompresses_each_client_first():
    """aggregate(states) = aggregate_var over the clients' decompressed variables; a client that
    kept a variable in FP32 contributes its precise values (Sec. 2.5)."""
    rng = np.random.default_rng(11)
    numel = [300, 17, 1000]
    base = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in numel]
    sels = [[True, False, True], [False, False, True], [True, True, False]]
    states = [orc.compress([p + np.float32(0.01 * k) for p in base], sel, 5, 2) for k, sel in enumerate(sels)]
    got = orc.aggregate(states)
    for i, n in enumerate(numel):
        xs = []
        for st in states:
            xs.append(orc.decompress_var(st["packed"][i], n, 5, 2, st["s"][i], st["b"][i]) if st["sel"][i]
                      else st["fp32"][i])
        want = xs[0].copy()
        for x in xs[1:]:
            want = want + x
        assert np.array_equal(got[i], want / np.float32(3))
    assert np.array_equal(states[1]["fp32"][0], base[0] + np.float32(0.01))


def test_two_stage_mean_is_sum_then_one_division():
    """Per-holder sums in client order, holders in order, one rounded division: exact rationals;
    one holder alone is the plain mean; the result stays within the stated bound of it."""
    rng = np.random.default_rng(21)
    n = 50
    xs = [(rng.standard_normal(n) * 10.0 ** rng.integers(-2, 2)).astype(np.float32) for _ in range(7)]
    groups = [xs[:3], xs[3:5], xs[5:]]
    got = orc.divide_var(orc.sum_var([orc.sum_var(g) for g in groups]), 7)
    for e in range(n):
        parts = []
        for g in groups:
            acc = np.float32(g[0][e])
            for x in g[1:]:
                acc = f32_round(Fraction(float(acc)) + Fraction(float(x[e])))
            parts.append(acc)
        tot = parts[0]
        for p in parts[1:]:
            tot = f32_round(Fraction(float(tot)) + Fraction(float(p)))
        assert got[e] == f32_round(Fraction(float(tot)) / 7)
    assert np.array_equal(orc.divide_var(orc.sum_var(xs), 7), orc.aggregate_var(xs))
    bound = 6 * 2.0 ** -24 * np.sum(np.abs(xs), axis=0) / 7 + 2.0 ** -24 * np.abs(orc.aggregate_var(xs))
    assert np.all(np.abs(got.astype(np.float64) - orc.aggregate_var(xs)) <= 2 * bound)


def test_sum_continued_batch_after_batch_is_the_one_pass_sum():
    """A sum that starts from the sum so far and adds the next batch of clients in order makes the
    additions of one pass over all clients, in the same order: forty clients in batches of 16, 16
    and 8 give the one-pass sum and mean bit for bit (the first element checked in exact rationals)."""
    rng = np.random.default_rng(33)
    n = 64
    xs = [(rng.standard_normal(n) * 10.0 ** rng.integers(-3, 3)).astype(np.float32) for _ in range(40)]
    run = orc.sum_var(xs[:16])
    run = orc.sum_var([run] + xs[16:32])
    run = orc.sum_var([run] + xs[32:])
    assert np.array_equal(run.view(np.uint32), orc.sum_var(xs).view(np.uint32))
    assert np.array_equal(orc.divide_var(run, 40).view(np.uint32), orc.aggregate_var(xs).view(np.uint32))
    acc = np.float32(xs[0][0])
    for x in xs[1:]:
        acc = f32_round(Fraction(float(acc)) + Fraction(float(x[0])))
    assert run[0] == acc

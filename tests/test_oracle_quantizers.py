"""Pins for the oracle's quantizers against exact rational arithmetic and the closed forms of Sec. 3.2.2."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2105_13890_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")


def golden(kind):
    out = []
    for line in open(GOLD):
        line = line.strip()
        if line and not line.startswith("#") and line.split()[0] == kind:
            out.append(line.split()[1:])
    assert out
    return out


def exact_round(fr: Fraction) -> int:
    # Python rounds a Fraction to the nearest integer with ties to even.
    return round(fr)


def test_rne_shr_matches_exact_rationals():
    for s in range(0, 13):
        for a in range(-3000, 3001):
            assert oracle.rne_shr(a, s) == exact_round(Fraction(a, 2**s)), (a, s)
    r = synth.rng(1, 1)
    for _ in range(20000):
        a = int(r.integers(-2**40, 2**40))
        s = int(r.integers(0, 45))
        assert oracle.rne_shr(a, s) == exact_round(Fraction(a, 2**s))


def test_rne_shr_ties_go_to_even_and_negative_shift_multiplies():
    assert [oracle.rne_shr(a, 1) for a in (1, 3, 5, -1, -3, -5)] == [0, 2, 2, 0, -2, -2]
    assert oracle.rne_shr(64, 7) == 0 and oracle.rne_shr(192, 7) == 2 and oracle.rne_shr(-64, 7) == 0
    assert oracle.rne_shr(-5, -3) == -40 and oracle.rne_shr(7, 0) == 7
    assert oracle.rne_shr(10**15, 70) == 0


def test_q_is_identity_on_its_grid_and_matches_closed_form():
    (k, den), = golden("q_grid")
    den = int(den)
    for j in range(-1000, 1001):
        assert oracle.q_code(j / den) == j
    assert oracle.q_code(0.3) == 38  # 0.3 * 128 = 38.4
    assert oracle.q_code(-0.3) == -38
    assert oracle.q_code(0.5 / den) == 0 and oracle.q_code(1.5 / den) == 2  # ties to even
    xs = np.sort(synth.normal_f32(2000, 3, 0, std=2.0))
    codes = [oracle.q_code(float(x)) for x in xs]
    assert all(b >= a for a, b in zip(codes, codes[1:]))  # monotone
    for x in xs[:300]:
        assert oracle.q_code(float(x)) == exact_round(Fraction(float(x)) * den)
        assert oracle.q_code(float(-x)) == -oracle.q_code(float(x))  # odd symmetry


def test_cq_range_and_saturation():
    (k, lo, hi), = golden("cq_bound")
    lo, hi = int(lo), int(hi)
    assert oracle.cq_code(1.0) == hi and oracle.cq_code(-1.0) == lo
    assert oracle.cq_code(55.0) == hi and oracle.cq_code(-55.0) == lo
    xs = synth.normal_f32(5000, 4, 0, std=1.0)
    codes, p, flag = oracle.quantize_f32(oracle.MODE_CQ, xs)
    assert p == -7 and flag == 0
    assert codes.min() >= lo and codes.max() <= hi and codes.min() == lo and codes.max() == hi
    inside = np.abs(xs) < 0.99
    q, _, _ = oracle.quantize_f32(oracle.MODE_Q, xs)
    assert np.array_equal(q[inside], codes[inside])
    assert q.max() > hi  # Q itself is unclamped


def brute_round_log2(m: Fraction) -> int:
    # the unique integer t with 2^(t-1/2) <= m < 2^(t+1/2), i.e. 2^(2t-1) <= m^2 < 2^(2t+1)
    t = -200
    sq = m * m
    while not (Fraction(2) ** (2 * t - 1) <= sq < Fraction(2) ** (2 * t + 1)):
        t += 1
        assert t < 200
    return t


def brute_sq(vals, p_a):
    m = max(abs(Fraction(v) * Fraction(2) ** p_a) for v in vals)
    t = brute_round_log2(m)
    scale = Fraction(2) ** t
    codes = []
    for v in vals:
        x = Fraction(v) * Fraction(2) ** p_a / scale
        codes.append(max(-127, min(127, exact_round(x * 128))))
    return codes, t - 7


def test_round_log2_matches_inequality_definition_and_float_log():
    for m in list(range(1, 3000)) + [2**31 - 1, 2**31, 2**32 + 5, 3037000499, 3037000500, 2**62 + 12345]:
        t = oracle.round_log2(m)
        assert t == brute_round_log2(Fraction(m)), m
        frac = math.log2(m) - math.floor(math.log2(m))
        if abs(frac - 0.5) > 1e-6:
            assert t == round(math.log2(m))
    # just below / above sqrt(2) * 2^f
    assert oracle.round_log2(90) == 6 and oracle.round_log2(91) == 7
    assert oracle.round_log2(181) == 7 and oracle.round_log2(182) == 8


def test_sq_int_matches_formula_in_exact_arithmetic():
    r = synth.rng(5, 0)
    for trial in range(300):
        n = int(r.integers(1, 9))
        mag = int(r.integers(1, 40))
        vals = [int(v) for v in r.integers(-2**mag, 2**mag + 1, size=n)]
        p_a = int(r.integers(-30, 5))
        codes, p_out, z = oracle.sq_int(np.array(vals), p_a)
        if all(v == 0 for v in vals):
            assert z == 1 and p_out == p_a and not codes.any()
            continue
        want, want_p = brute_sq(vals, p_a)
        assert z == 0 and list(codes) == want and p_out == want_p, (vals, p_a)


def test_sq_invariants():
    r = synth.rng(6, 0)
    a = r.integers(-50000, 50001, size=4096)
    codes, p, z = oracle.sq_int(a, -14)
    assert z == 0 and 91 <= np.abs(codes).max() <= 127 and codes.min() >= -127
    # power-of-two equivariance: SQ(2^t x) = 2^t SQ(x)
    for t in (1, 5, 11):
        c2, p2, _ = oracle.sq_int(a * 2**t, -14)
        assert np.array_equal(c2, codes) and p2 == p + t
        c3, p3, _ = oracle.sq_int(a, -14 + t)
        assert np.array_equal(c3, codes) and p3 == p + t
    # idempotence: SQ(SQ(x)) = SQ(x)
    c4, p4, _ = oracle.sq_int(codes.astype(np.int64), p)
    assert np.array_equal(c4, codes) and p4 == p
    # the scale is the power of two nearest (in log) to the maximum
    m = Fraction(int(np.abs(a).max())) * Fraction(2) ** -14
    assert Fraction(2) ** (2 * (p + 7) - 1) <= m * m < Fraction(2) ** (2 * (p + 7) + 1)
    # clipping happens when max/scale > 127/128 (log-rounding lets it reach sqrt 2)
    c5, p5, _ = oracle.sq_int(np.array([181, 100, -181]), 0)
    assert p5 == 0 and list(c5) == [127, 100, -127]
    c6, p6, _ = oracle.sq_int(np.array([182, 100, -182]), 0)
    assert p6 == 1 and list(c6) == [91, 50, -91]
    z0 = oracle.sq_int(np.zeros(5, dtype=np.int64), -9)
    assert z0[2] == 1 and z0[1] == -9 and not z0[0].any()


def test_sq_float_agrees_with_integer_path_and_formula():
    r = synth.rng(7, 0)
    ints = r.integers(-3000, 3001, size=777)
    cf, pf, zf = oracle.quantize_f32(oracle.MODE_SQ, ints.astype(np.float32))
    ci, pi, zi = oracle.sq_int(ints, 0)
    assert np.array_equal(cf, ci) and pf == pi and zf == zi == 0
    for trial in range(100):
        x = synth.normal_f32(int(r.integers(1, 7)), 8, trial, std=float(10.0 ** r.uniform(-6, 6)))
        if not np.any(x):
            continue
        vals = [Fraction(float(v)) for v in x]
        want, want_p = brute_sq(vals, 0)
        c, p, z = oracle.quantize_f32(oracle.MODE_SQ, x)
        assert list(c) == want and p == want_p and z == 0
    assert oracle.quantize_f32(oracle.MODE_SQ, np.array([1.0, np.inf], dtype=np.float32))[2] == -1
    assert oracle.quantize_f32(oracle.MODE_SQ, np.zeros(3, dtype=np.float32))[2] == 1


def test_scalar_init_codes():
    (g, b), = golden("scalar_init")
    assert oracle.q_code(1.0) == int(g) and oracle.q_code(0.0) == int(b)

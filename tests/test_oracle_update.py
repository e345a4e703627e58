"""Pins for the 8-bit update: invariants and exact-arithmetic brute force (semantics themselves: parity unpinned)."""
from fractions import Fraction as Fr

import numpy as np

import oracle
from paper_2105_13890_b200 import synth


def test_zero_gradient_leaves_weights_unchanged():
    w = synth.int8_uniform(500, 30, 0)
    new, p_u, z = oracle.update(w, np.zeros(500, dtype=np.int8), -10, 3, -4)
    assert z == 1 and np.array_equal(new, w)


def test_unit_mantissa_keeps_gradient_codes():
    """lr = 2^e only moves the exponent: SQ is idempotent and power-of-two equivariant (Sec. 3.2.2)."""
    g, p_g, _ = oracle.sq_int(synth.rng(31, 0).integers(-9000, 9001, size=400), 0)
    w = np.zeros(400, dtype=np.int32)
    new, p_u, _ = oracle.update(w, g.astype(np.int8), p_g, 1, -2, lo=-10**6, hi=10**6)
    assert p_u == p_g - 2
    d = p_u + 7
    assert d >= 0
    assert np.array_equal(new, -(g.astype(np.int64) << d))


def brute_update(theta, g, p_g, lr_mant, lr_exp, lo, hi):
    lr = Fr(lr_mant) * Fr(2) ** lr_exp
    vals = [lr * Fr(int(v)) * Fr(2) ** p_g for v in g]
    m = max(abs(v) for v in vals)
    if m == 0:
        return list(theta)
    t = -300
    while not (Fr(2) ** (2 * t - 1) <= m * m < Fr(2) ** (2 * t + 1)):
        t += 1
    scale = Fr(2) ** t
    out = []
    for th, v in zip(theta, vals):
        u = scale * Fr(max(-127, min(127, round(v / scale * 128))), 128)   # Q_u = SQ(lr * g)
        new = Fr(int(th), 128) - u
        out.append(max(lo, min(hi, round(new * 128))))                      # parameter quantizer on the 2^-7 grid
    return out


def test_update_matches_exact_rational_arithmetic_across_alignments():
    r = synth.rng(32, 0)
    for trial in range(400):
        n = int(r.integers(1, 10))
        g = r.integers(-127, 128, size=n).astype(np.int8)
        theta = r.integers(-127, 128, size=n).astype(np.int32)
        p_g = int(r.integers(-24, 2))
        lr_mant = int(r.integers(1, 256))
        lr_exp = int(r.integers(-12, 3))
        new, _, _ = oracle.update(theta, g, p_g, lr_mant, lr_exp)
        assert list(new) == brute_update(theta, g, p_g, lr_mant, lr_exp, -127, 127), (trial, g, theta, p_g, lr_mant, lr_exp)


def test_range_is_preserved_and_scalars_use_int16_range():
    g = np.array([127, -127], dtype=np.int8)
    new, _, _ = oracle.update(np.array([-120, 120]), g, 0, 1, 0)
    assert list(new) == [-127, 127]
    new, _, _ = oracle.update(np.array([128]), np.array([-100], dtype=np.int8), -7, 1, 0, lo=-32768, hi=32767)
    assert list(new) == [228]


def test_stochastic_rounding_is_unbiased_and_counter_based():
    g = np.full(20000, 100, dtype=np.int8)
    g[0] = 127
    theta = np.zeros(20000, dtype=np.int32)
    # u codes = g codes at exponent -10: three bits below the weight grid
    new, p_u, _ = oracle.update(theta, g, -10, 1, 0, stochastic=True, seed=9, step=4, tensor_id=2)
    assert p_u == -10
    assert set(np.unique(new[1:])) <= {-12, -13}
    assert abs(-new[1:].mean() - 100 / 8) < 0.02
    again, _, _ = oracle.update(theta, g, -10, 1, 0, stochastic=True, seed=9, step=4, tensor_id=2)
    other, _, _ = oracle.update(theta, g, -10, 1, 0, stochastic=True, seed=9, step=5, tensor_id=2)
    assert np.array_equal(new, again) and not np.array_equal(new, other)
    rne, _, _ = oracle.update(theta, g, -10, 1, 0)
    assert set(np.unique(rne[1:])) == {-12}  # 12.5 ties to even
    assert oracle.update_hash(1, 2, 3, 4) != oracle.update_hash(1, 2, 3, 5)


# ------------------------------------------------------------------ other update widths (the 24-bit update the paper compares with)

def brute_update_k(theta, g, p_g, lr_mant, lr_exp, k_u, k_m):
    lr = Fr(lr_mant) * Fr(2) ** lr_exp
    vals = [lr * Fr(int(v)) * Fr(2) ** p_g for v in g]
    m = max(abs(v) for v in vals)
    if m == 0:
        return list(theta)
    t = -300
    while not (Fr(2) ** (2 * t - 1) <= m * m < Fr(2) ** (2 * t + 1)):
        t += 1
    scale, lu, lm = Fr(2) ** t, 2 ** (k_u - 1), 2 ** (k_m - 1)
    out = []
    for th, v in zip(theta, vals):
        u = scale * Fr(max(-(lu - 1), min(lu - 1, round(v / scale * lu))), lu)   # SQ(lr g, k_u)
        new = Fr(int(th), lm) - u
        out.append(max(-(lm - 1), min(lm - 1, round(new * lm))))               # CQ(., k_m)
    return out


def test_wide_update_matches_exact_rational_arithmetic():
    r = synth.rng(33, 0)
    for k_u, k_m in ((8, 8), (16, 16), (24, 24), (8, 24), (16, 8)):
        for trial in range(150):
            n = int(r.integers(1, 8))
            g = r.integers(-127, 128, size=n).astype(np.int8)
            lim = 2 ** (k_m - 1) - 1
            theta = r.integers(-lim, lim + 1, size=n).astype(np.int32)
            p_g, lr_mant, lr_exp = int(r.integers(-24, 2)), int(r.integers(1, 256)), int(r.integers(-12, 3))
            new, w8, _, _ = oracle.update_k(theta, g, p_g, lr_mant, lr_exp, k_u, k_m)
            assert list(new) == brute_update_k(theta, g, p_g, lr_mant, lr_exp, k_u, k_m), (k_u, k_m, trial)
            assert list(w8) == [max(-127, min(127, round(Fr(int(v), 2 ** (k_m - 8))))) for v in new]


def test_eight_bit_case_of_the_wide_update_is_the_paper_update():
    r = synth.rng(34, 0)
    g = r.integers(-127, 128, size=300).astype(np.int8)
    theta = r.integers(-127, 128, size=300).astype(np.int32)
    for stochastic in (False, True):
        a, _, pa, _ = oracle.update_k(theta, g, -11, 37, -3, 8, 8, stochastic=stochastic, seed=5, step=2, tensor_id=1)
        b, pb, _ = oracle.update(theta, g, -11, 37, -3, stochastic=stochastic, seed=5, step=2, tensor_id=1)
        assert np.array_equal(a, b) and pa == pb


def test_generic_width_scale_quantizer_invariants():
    a = synth.rng(35, 0).integers(-10**9, 10**9, size=500)
    for k in (4, 8, 16, 24):
        c, p, _ = oracle.sq_int_k(a, -30, k)
        lim = 2 ** (k - 1) - 1
        assert np.abs(c).max() <= lim and np.abs(c).max() >= (lim + 1) / np.sqrt(2) - 1      # largest code in [2^(k-1)/sqrt 2, lim]
        c2, p2, _ = oracle.sq_int_k(a * 8, -30, k)                                            # power-of-two equivariance
        assert np.array_equal(c, c2) and p2 == p + 3
    c8, p8, _ = oracle.sq_int_k(a, -30, 8)
    ref, pr, _ = oracle.sq_int(a, -30)
    assert np.array_equal(c8, ref) and p8 == pr


def test_wide_master_copy_keeps_updates_the_eight_bit_update_rounds_away():
    """What the update width changes: steps far below the 8-bit weight grid vanish under nearest rounding with an
    8-bit master copy, but accumulate in a 24-bit one."""
    g = np.full(64, 100, dtype=np.int8)
    g[0] = 127
    th8, th24 = np.zeros(64, dtype=np.int32), np.zeros(64, dtype=np.int32)
    for _ in range(40):
        th8, _, _ = oracle.update(th8, g, -18, 1, 0)                     # u = 100 * 2^-18: a twentieth of a weight step
        th24, w24, _, _ = oracle.update_k(th24, g, -18, 1, 0, 24, 24)
    assert not th8.any()
    assert (th24[1:] == -40 * 100 * 2 ** 5).all() and (w24[1:] == -2).all()   # 40 * 100 * 2^-18 = 1.95 / 128 -> code -2

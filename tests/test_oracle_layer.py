"""Pins for the forward epilogue, the backward chain and the Fixup initialisation."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import ConvDesc
from paper_2105_13890_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")


def golden(kind):
    return [l.split()[1:] for l in open(GOLD) if l.strip() and not l.startswith("#") and l.split()[0] == kind]


def test_epilogue_at_initialisation_is_clamped_relu_of_x2():
    """gamma = 1 (code 128), biases 0, no shortcut: x5 = sat(max(x2, 0), 0, 127) (scalars as initialised, Sec. 3.2.3)."""
    A = synth.rng(20, 0).integers(-40000, 40001, size=(2, 4, 4, 8))
    x2, x5, mask = oracle.fwd_epilogue(A, 7, 128, 0)
    assert np.array_equal(x5, np.clip(x2, 0, 127).astype(np.int8))
    assert np.array_equal(mask, (x2 > 0).astype(np.uint8))
    assert np.array_equal(x2, np.array([oracle.rne_shr(int(a), 7) for a in A.ravel()]).reshape(A.shape))


def test_epilogue_chain_in_exact_rationals():
    """x5 = CQ(relu(Q(gamma) * Q(conv) + Q(b2) + shortcut)) evaluated with fractions (forward chain, Sec. 3.2.1)."""
    from fractions import Fraction as Fr

    r = synth.rng(21, 0)
    A = r.integers(-60000, 60001, size=64)
    sc = synth.int8_uniform(64, 21, 1)
    for gamma_c, b2_c, relu, use_sc in [(128, 0, True, False), (90, 5, True, True), (-37, -300, False, True), (700, 40, True, False)]:
        x2, x5, mask = oracle.fwd_epilogue(A, 7, gamma_c, b2_c, sc if use_sc else None, relu)
        for i in range(64):
            conv = Fr(int(A[i]), 2**14)
            q2 = Fr(round(conv * 128), 128)
            x4 = Fr(gamma_c, 128) * q2 + Fr(b2_c, 128) + (Fr(int(sc[i]), 128) if use_sc else 0)
            v = max(x4, 0) if relu else x4
            code = max(-127, min(127, round(v * 128)))
            assert x2[i] == q2 * 128 and x5[i] == code and mask[i] == (x4 > 0)


def test_epilogue_is_linear_in_b2_before_rounding_and_x2_saturates():
    A = np.array([5 * 128, -3 * 128, 2**30, -2**30])
    x2, x5, _ = oracle.fwd_epilogue(A, 7, 128, 0, None, False)
    assert list(x2) == [5, -3, 32767, -32768] and list(x5) == [5, -3, 127, -127]
    _, x5b, _ = oracle.fwd_epilogue(A, 7, 128, 10, None, False)
    assert list(x5b[:2]) == [15, 7]
    # network input at exponent p_in = -5: accumulator exponent -12, Q_a1 shift is 5
    x2c, _, _ = oracle.fwd_epilogue(np.array([32 * 9, 33]), 5, 128, 0)
    assert list(x2c) == [9, 1]


def test_layer_forward_with_identity_kernel_is_relu_of_x1():
    d = ConvDesc(1, 6, 6, 4, 4, 3, 3, 1, 1)
    x0 = (2 * synth.int8_uniform((1, 6, 6, 4), 22, 0, -50, 50)).astype(np.int8)  # even, so halving is exact
    w = np.zeros((4, 3, 3, 4), dtype=np.int8)
    for c in range(4):
        w[c, 1, 1, c] = 64  # 0.5; gamma = 2 (code 256) restores unit gain
    out = oracle.layer_forward(d, x0, -4, w, 256, 0)
    assert np.array_equal(out["x5"], np.clip(x0.astype(np.int64) - 4, 0, 127).astype(np.int8))


def test_backward_chain_equals_float_autograd_when_nothing_rounds():
    """With data on which no quantizer rounds or clips, the error chain and the gradients (Sec. 3.2.1) must equal
    autograd of the unquantized forward chain (straight-through estimator = identity)."""
    d = ConvDesc(2, 5, 5, 2, 3, 3, 3, 1, 1)
    r = synth.rng(23, 0)
    x0 = (16 * r.integers(-7, 8, size=(d.n, d.h, d.w, d.c_in))).astype(np.int8)
    w = (8 * r.integers(-3, 4, size=(d.c_out, d.kh, d.kw, d.c_in))).astype(np.int8)
    e0 = r.integers(-3, 4, size=(d.n, d.ho, d.wo, d.c_out)).astype(np.int8)
    e0.flat[0] = 3
    b1_c, gamma_c, b2_c, p0 = 16, 2 * 128, 64, -9
    fwd = oracle.layer_forward(d, x0, b1_c, w, gamma_c, b2_c)
    assert np.all(fwd["acc"] % 128 == 0)  # Q_a1 does not round here
    bwd = oracle.layer_backward(d, e0, p0, fwd["mask"], fwd["x2"], x0, b1_c, w, gamma_c)

    def t(a, perm=(0, 3, 1, 2)):
        return torch.from_numpy(np.ascontiguousarray(a)).to(torch.float64).permute(*perm).contiguous()

    x0f = (t(x0) / 128).requires_grad_(True)
    wf = (t(w) / 128).requires_grad_(True)
    b1 = torch.tensor(b1_c / 128, dtype=torch.float64, requires_grad=True)
    gam = torch.tensor(gamma_c / 128, dtype=torch.float64, requires_grad=True)
    b2 = torch.tensor(b2_c / 128, dtype=torch.float64, requires_grad=True)
    x1 = F.pad(x0f + b1, (1, 1, 1, 1))
    x2 = F.conv2d(x1, wf)
    x4 = gam * x2 + b2
    x5 = torch.relu(x4)
    x5.backward(t(e0) * 2.0**p0)

    def real(codes, p):
        return np.asarray(codes, dtype=np.float64) * 2.0**p

    assert np.array_equal(real(bwd["e4"], bwd["p4"]), x0f.grad.permute(0, 2, 3, 1).numpy())
    assert np.array_equal(real(bwd["g_w"], bwd["p_gw"]), wf.grad.permute(0, 2, 3, 1).numpy())
    # scalar gradients: the sums are exact; Q_g of a lone scalar may clip it (its max can exceed 127/128 of the scale)
    assert real(bwd["sum_e1"], p0) == b2.grad.item()
    assert real(bwd["sum_e1x2"], p0 - 7) == gam.grad.item()
    assert real(bwd["sum_e4"], bwd["p4"]) == b1.grad.item()
    for key, s, p in (("g_b2", bwd["sum_e1"], p0), ("g_gamma", bwd["sum_e1x2"], p0 - 7), ("g_b1", bwd["sum_e4"], bwd["p4"])):
        c, pp, _ = oracle.sq_int(np.array([s]), p)
        assert bwd[key] == (int(c[0]), pp)
        assert abs(real(*bwd[key]) - real(s, p)) <= abs(real(s, p)) * 0.30
    assert np.abs(bwd["e4"]).max() <= 127 and np.abs(bwd["g_w"]).max() <= 127


def test_error_prescale_pieces():
    e0 = np.array([10, -20, 30, -40, 50], dtype=np.int8)
    mask = np.array([1, 0, 1, 1, 0], dtype=np.uint8)
    x2 = np.array([3, 100, -2, 7, 9], dtype=np.int32)
    e3, p3, s1, s2, z = oracle.err_prescale(e0, -5, mask, x2, 64)
    # gamma * e1 = [640, 0, 1920, -2560, 0] at 2^-12; max 2560 -> t = 11, shift 4
    assert list(e3) == [40, 0, 120, -127, 0] and p3 == -12 + 4 and z == 0  # -160 clips to -127
    assert s1 == 10 + 30 - 40 and s2 == 30 - 60 - 280


def test_fixup_alpha_and_traces_match_closed_forms():
    for L, m, val in golden("alpha"):
        assert oracle.fixup_alpha(int(L), int(m)) == pytest.approx(float(val), rel=1e-15)
    for L, m, val in golden("branch_layer_trace"):
        assert oracle.fixup_alpha(int(L), int(m)) ** 2 == pytest.approx(float(val), rel=1e-14)
    for L, m, val in golden("branch_trace"):
        assert oracle.fixup_alpha(int(L), int(m)) ** (2 * int(m)) == pytest.approx(float(val), rel=1e-14)


def test_fixup_weight_statistics_and_variance_propagation():
    """Branch layers carry variance ratio L^(-1/(m-1)) each and L^(-m/(m-1)) per branch (Sec. 4, Fixup analysis)."""
    L, m, c, k = 8, 2, 32, 3
    fan_in = c * k * k
    z = synth.normal_f64((c, k, k, c), 24, 0)
    w = oracle.fixup_weights_f32(z, fan_in, L, m)
    assert w.std() == pytest.approx(np.sqrt(2.0 / fan_in) * L ** (-1.0 / (2 * m - 2)), rel=0.03)
    w_main = oracle.fixup_weights_f32(z, fan_in, L, m, in_branch=False)
    assert w_main.std() == pytest.approx(np.sqrt(2.0 / fan_in), rel=0.03)
    x = torch.from_numpy(synth.normal_f64((8, c, 16, 16), 24, 1))
    ratios = []
    h = x
    for layer in range(m):
        wz = oracle.fixup_weights_f32(synth.normal_f64((c, k, k, c), 24, 10 + layer), fan_in, L, m)
        wt = torch.from_numpy(wz).to(torch.float64).permute(0, 3, 1, 2)
        y = F.conv2d(torch.relu(h), wt, padding=1)
        ratios.append((y.var() / h.var()).item())
        h = y
    (_, _, per_layer), = [g for g in golden("branch_layer_trace") if g[0] == "8"]
    (_, _, branch), = [g for g in golden("branch_trace") if g[0] == "8"]
    for rr in ratios:
        assert rr == pytest.approx(float(per_layer), rel=0.12)
    assert (h.var() / x.var()).item() == pytest.approx(float(branch), rel=0.2)


def test_q_w_of_fixup_weights_stays_in_range_with_expected_code_spread():
    z = synth.normal_f64((16, 3, 3, 16), 25, 0)
    w = oracle.fixup_weights_f32(z, 144, 1, 2, in_branch=False)
    codes = oracle.q_w(w)
    assert codes.dtype == np.int8 and codes.min() >= -127
    assert codes.std() == pytest.approx(128 * np.sqrt(2 / 144), rel=0.06)

"""Pins of the oracle's network glue (pooling, error join, float head, block composition).

The paper fixes none of these conventions, so they are pinned by what mathematics and library routines fix:
library pooling and autograd on float64 copies, exact rational arithmetic, closed forms of softmax cross-entropy,
and -- for the composition of a whole residual block -- float autograd on data where no quantizer rounds.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import ConvDesc
from oracle import network as N
from paper_2105_13890_b200 import synth


def test_maxpool_matches_library_pooling_and_routes_to_first_maximum():
    x = synth.int8_uniform((2, 9, 7, 5), 41, 0, -20, 20)   # small range: many ties
    y, idx = oracle.maxpool_fwd(x, 3, 2, 1)
    ref = F.max_pool2d(torch.from_numpy(x).double().permute(0, 3, 1, 2), 3, 2, 1).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(y.astype(np.float64), ref)
    n, h, w, c = x.shape
    for b, oy, ox, ch in [(0, 0, 0, 0), (1, 4, 3, 4), (0, 2, 1, 3), (1, 0, 3, 1)]:
        first = None
        for kh in range(3):
            for kw in range(3):
                iy, ix = oy * 2 + kh - 1, ox * 2 + kw - 1
                if 0 <= iy < h and 0 <= ix < w and x[b, iy, ix, ch] == y[b, oy, ox, ch] and first is None:
                    first = ((b * h + iy) * w + ix) * c + ch
        assert idx[b, oy, ox, ch] == first


def test_maxpool_backward_matches_autograd_when_maxima_are_unique():
    r = synth.rng(42, 0)
    x = r.permutation(2 * 8 * 8 * 3)[: 2 * 8 * 8 * 3].reshape(2, 8, 8, 3) % 120   # few ties
    x = (x - 60).astype(np.int8)
    xt = torch.from_numpy(x).double().permute(0, 3, 1, 2).requires_grad_(True)
    # make maxima unique by a tiny position-dependent offset that does not change the integer winner order
    eps = torch.arange(xt.shape[2] * xt.shape[3], dtype=torch.float64).reshape(1, 1, xt.shape[2], xt.shape[3]) * 1e-9
    yt = F.max_pool2d(xt - eps, 3, 2, 1)
    e = synth.normal_codes(tuple(yt.permute(0, 2, 3, 1).shape), 43, 0)
    yt.backward(torch.from_numpy(e).double().permute(0, 3, 1, 2))
    _, idx = oracle.maxpool_fwd(x, 3, 2, 1)
    S = oracle.maxpool_bwd(e, idx, x.shape)
    # the offset grows along the (kh, kw) scan order, so among equal codes the earliest position wins in both
    assert np.array_equal(S.astype(np.float64), xt.grad.permute(0, 2, 3, 1).numpy())
    assert S.sum() == e.astype(np.int64).sum()


def test_avgpool_sum_is_the_plain_sum():
    x = synth.int8_uniform((3, 4, 5, 6), 44, 0)
    assert np.array_equal(oracle.avgpool_sum(x), x.astype(np.int64).sum(axis=(1, 2)))


@pytest.mark.parametrize("pa,pb", [(-9, -9), (-12, -7), (-7, -15), (-3, -40), (-50, -10)])
def test_error_join_is_the_exact_sum_at_the_smaller_exponent(pa, pb):
    a = synth.normal_codes(200, 45, 0)
    b = synth.normal_codes(200, 45, 1)
    mask = synth.bits(200, 45, 2)
    for m in (None, mask):
        S, p = oracle.join(a, pa, b, pb, m)
        bm = b if m is None else b * m.astype(np.int8)
        if abs(pa - pb) <= 31:
            assert p == min(pa, pb)
            for i in range(0, 200, 7):
                assert Fraction(int(S[i])) * Fraction(2) ** p == Fraction(int(a[i])) * Fraction(2) ** pa + Fraction(int(bm[i])) * Fraction(2) ** pb
        elif pa > pb:   # b is more than 31 octaves below a: dropped
            assert p == pa and np.array_equal(S, a.astype(np.int64))
        else:
            assert p == pb and np.array_equal(S, bm.astype(np.int64))


def test_own_exp_is_accurate_and_exact_at_zero():
    assert oracle.expf(0.0) == 1.0
    xs = np.concatenate([np.linspace(-87, 0, 3001), np.linspace(0, 20, 500), -np.logspace(-8, 1.9, 300)]).astype(np.float32)
    worst = max(abs(oracle.expf(float(v)) / math.exp(float(v)) - 1.0) for v in xs)
    assert worst < 2.5e-7
    vals = [oracle.expf(float(v)) for v in np.linspace(-30, 0, 4000).astype(np.float32)]
    assert all(b >= a for a, b in zip(vals, vals[1:]))   # monotone
    assert oracle.expf(-100.0) == 0.0


def test_float_head_matches_a_float64_reference_and_closed_forms():
    n, c, classes, hw = 8, 32, 10, 16
    sums = synth.rng(46, 0).integers(0, 127 * hw, size=(n, c)).astype(np.int64)
    W = (synth.normal_f32((classes, c), 46, 1) * 0.2).astype(np.float32)
    bias = (synth.normal_f32((classes,), 46, 2) * 0.1).astype(np.float32)
    labels = synth.labels(n, classes, 46, 3).astype(np.int32)
    lr = 2.0 ** -5
    W0, b0 = W.copy(), bias.copy()
    loss, dpooled, logits = oracle.head(sums, hw, W, bias, labels, lr)
    pooled = torch.tensor(sums / 128.0 / hw, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W0, dtype=torch.float64, requires_grad=True)
    bt = torch.tensor(b0, dtype=torch.float64, requires_grad=True)
    lt = pooled @ Wt.t() + bt
    ref = F.cross_entropy(lt, torch.from_numpy(labels.astype(np.int64)))
    ref.backward()
    assert np.allclose(logits, lt.detach().numpy(), rtol=2e-6, atol=2e-6)
    assert loss == pytest.approx(ref.item(), rel=2e-6)
    assert np.allclose(dpooled, pooled.grad.numpy(), rtol=2e-5, atol=1e-8)
    assert np.allclose(W, W0 - lr * Wt.grad.numpy(), rtol=1e-6, atol=1e-7)
    assert np.allclose(bias, b0 - lr * bt.grad.numpy(), rtol=1e-6, atol=1e-7)
    # uniform logits: the loss is ln(classes) and the gradient of the pooled activations vanishes with zero weights
    Wz, bz = np.zeros((classes, c), dtype=np.float32), np.zeros(classes, dtype=np.float32)
    loss0, dp0, lg0 = oracle.head(sums, hw, Wz, bz, labels, 0.0)
    assert loss0 == pytest.approx(math.log(classes), rel=1e-6) and not dp0.any() and not lg0.any()


def _tiny_net(proj: bool, seed: int):
    """One residual block behind a first layer, with data on which no quantizer rounds: activations multiples of 16,
    weights multiples of 16 (unit B: two taps of +-64 per output channel), scalars multiples of 16."""
    r = synth.rng(seed, 0)
    c0, c1 = 2, (4 if proj else 2)
    stride = 2 if proj else 1
    units = [N.Unit("stem", ConvDesc(1, 6, 6, 2, c0, 1, 1, 1, 0), 2, "stem", in_branch=False),
             N.Unit("a", ConvDesc(1, 6, 6, c0, c1, 3, 3, stride, 1), c0, "a")]
    blk = N.Block(1, 2)
    if proj:
        units.append(N.Unit("proj", ConvDesc(1, 6, 6, c0, c1, 1, 1, stride, 0), c0, "proj", relu=False, in_branch=False))
        blk = N.Block(1, 3, 2)
    h1 = 3 if proj else 6
    units.append(N.Unit("b", ConvDesc(1, h1, h1, c1, c1, 3, 3, 1, 1), c1, "b"))
    net = N.Net(units, [blk], None, 10, L=1, m=2)
    for u in units:
        d = u.d
        u.w = np.zeros((d.c_out, d.kh, d.kw, d.c_in), dtype=np.int8)
    units[0].w[0, 0, 0, 0] = units[0].w[1, 0, 0, 1] = 64           # first layer: half of the input
    ua, ub = units[blk.a], units[blk.b]
    ua.w[...] = (16 * r.integers(-1, 2, size=ua.w.shape) * (r.random(size=ua.w.shape) < 0.4)).astype(np.int8)
    for oc in range(c1):
        ub.w[oc, 1, 1, oc] = 64 * int(r.choice([-1, 1]))
        ub.w[oc, 0, 1, (oc + 1) % c1] = 64
    if proj:
        units[blk.proj].w[...] = (32 * r.integers(-1, 2, size=units[blk.proj].w.shape)).astype(np.int8)
    ua.b1, ua.b2 = 16, 32
    ub.b1, ub.gamma, ub.b2 = -16, 256, 16
    units[0].b2 = 16
    return net, blk


@pytest.mark.parametrize("proj", [False, True], ids=["identity_shortcut", "projection_shortcut"])
def test_block_composition_equals_float_autograd_when_nothing_rounds(proj):
    """Forward chain, shortcut, error join and every gradient of one residual block against autograd of the
    unquantized float network (straight-through estimator = identity), on data where no quantizer rounds or clips.
    Seeds are tried until the data meets that condition at every quantizer; the condition itself is asserted."""
    def real(codes, p):
        return np.asarray(codes, dtype=np.float64) * 2.0 ** p

    def t(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(torch.float64).permute(0, 3, 1, 2).contiguous()

    found = 0
    for seed in range(60, 4000):
        net, blk = _tiny_net(proj, seed)
        units = net.units
        r = synth.rng(seed, 1)
        x_in = (32 * r.integers(0, 4, size=(1, 6, 6, 2))).astype(np.int8)
        fw, x0s, x, _ = N.forward_trunk(net, x_in, -7)
        e_out = r.integers(-3, 4, size=x.shape).astype(np.int8)
        e_out.flat[0] = 3
        p_out = -9
        bw, grads, scal, _ = N.backward_trunk(net, fw, x0s, None, e_out, p_out)
        ua, ub = units[blk.a], units[blk.b]
        fa, fb, ba, bb = fw[blk.a], fw[blk.b], bw[blk.a], bw[blk.b]
        # nothing rounded or clipped anywhere?
        exact = all(np.all(f["acc"] % 128 == 0) for f in fw.values())
        exact &= all(np.abs(f["x5"]).max() < 127 for f in fw.values()) and np.all(fb["x2"] * ub.gamma % 128 == 0)
        checks = [(bb["e4"], bb["p4"], bb["dgrad_acc"], bb["p3"] - 7), (bb["g_w"], bb["p_gw"], bb["wgrad_acc"], bb["p3"] - 7),
                  (ba["e4"], ba["p4"], ba["dgrad_acc"], ba["p3"] - 7), (ba["g_w"], ba["p_gw"], ba["wgrad_acc"], ba["p3"] - 7),
                  (ba["join"], ba["p_join"], ba["join_acc"], ba["join_acc_exp"])]
        if proj:
            bp = bw[blk.proj]
            checks += [(bp["e4"], bp["p4"], bp["dgrad_acc"], bp["p3"] - 7), (bp["g_w"], bp["p_gw"], bp["wgrad_acc"], bp["p3"] - 7)]
        exact &= all(np.array_equal(real(c, p), real(acc, pacc)) for c, p, acc, pacc in checks)
        exact &= np.array_equal(real(bb["e3"], bb["p3"]), real(e_out.astype(np.int64) * fb["mask"] * ub.gamma, p_out - 7))
        exact &= np.array_equal(real(ba["e3"], ba["p3"]), real(bb["e4"].astype(np.int64) * fa["mask"] * 128, bb["p4"] - 7))
        if not exact or not fb["mask"].any() or not ba["join"].any():
            continue
        found += 1
        # the same block in float64 with autograd
        xb = t(fw[0]["x5"]) / 128
        xb.requires_grad_(True)
        wa, wb = (t(ua.w) / 128).requires_grad_(True), (t(ub.w) / 128).requires_grad_(True)
        par = {k: torch.tensor(v / 128, dtype=torch.float64, requires_grad=True)
               for k, v in (("b1a", ua.b1), ("b2a", ua.b2), ("b1b", ub.b1), ("gb", ub.gamma), ("b2b", ub.b2))}
        st = ua.d.stride
        a5 = torch.relu(F.conv2d(F.pad(xb + par["b1a"], (1, 1, 1, 1)), wa, stride=st) + par["b2a"])
        if proj:
            wp = (t(units[blk.proj].w) / 128).requires_grad_(True)
            short = F.conv2d(xb + par["b1a"], wp, stride=st)
        else:
            short = xb
        y5 = torch.relu(par["gb"] * F.conv2d(F.pad(a5 + par["b1b"], (1, 1, 1, 1)), wb) + par["b2b"] + short)
        assert np.array_equal(fb["x5"].astype(np.float64) / 128, y5.detach().permute(0, 2, 3, 1).numpy())   # forward chain
        y5.backward(t(e_out) * 2.0 ** p_out)
        assert np.array_equal(real(ba["join"], ba["p_join"]), xb.grad.permute(0, 2, 3, 1).numpy())          # block input error
        assert np.array_equal(real(bb["g_w"], bb["p_gw"]), wb.grad.permute(0, 2, 3, 1).numpy())
        assert np.array_equal(real(ba["g_w"], ba["p_gw"]), wa.grad.permute(0, 2, 3, 1).numpy())
        if proj:
            assert np.array_equal(real(bw[blk.proj]["g_w"], bw[blk.proj]["p_gw"]), wp.grad.permute(0, 2, 3, 1).numpy())
        sums = {(units[i].name, which): real(total, p) for i, which, total, p in scal}
        assert sums[("b", "b1")] == par["b1b"].grad.item() and sums[("b", "b2")] == par["b2b"].grad.item()
        assert sums[("b", "gamma")] == par["gb"].grad.item()
        assert sums[("a", "b2")] == par["b2a"].grad.item() and sums[("a", "b1")] == par["b1a"].grad.item()
        if found == 3:
            break
    assert found >= 1


def test_closed_loop_step_runs_and_updates_every_parameter_kind():
    net = N.resnet20(2)
    N.init(net, lambda s, st: synth.normal_f64(s, 7, st), lambda s, st: synth.normal_f32(s, 7, st), b1=-2, gamma=118, b2=3)
    before = [(u.w.copy(), u.b1, u.gamma, u.b2) for u in net.units]
    W0 = net.W.copy()
    img, labels = synth.normal_f32((2, 32, 32, 3), 7, 0), synth.labels(2, 10, 7, 1)
    log = N.train_step(net, img, labels, 3, -4, 2.0 ** -6)
    assert 1.0 < log["head"]["loss"] < 4.0                       # near ln(10) at initialisation
    assert any(not np.array_equal(u.w, b[0]) for u, b in zip(net.units, before))
    assert any((u.b1, u.gamma, u.b2) != b[1:] for u, b in zip(net.units, before))
    assert not np.array_equal(net.W, W0)
    for u in net.units:                                           # fixed scalars stay fixed
        if u.role != "b":
            assert u.gamma == 128
        if u.role == "proj":
            assert u.b2 == 0
        if u.role == "stem":
            assert u.b1 == 0
    # every unit's e0 is its successor's error: unit A of the last block receives e4 of unit B
    blk = net.blocks[-1]
    ua, ub = net.units[blk.a], net.units[blk.b]
    e3a, p3a, _, _, _ = oracle.err_prescale(log[ub.name]["bwd"]["e4"], log[ub.name]["bwd"]["p4"], log[ua.name]["fwd"]["mask"], None, 128)
    assert np.array_equal(e3a, log[ua.name]["bwd"]["e3"]) and p3a == log[ua.name]["bwd"]["p3"]

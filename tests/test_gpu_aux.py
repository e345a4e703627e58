"""The glue entry points (eoq_aux_*) one by one against the oracle, element by element: pooling over several window
geometries and ragged image sizes, the error join over exponent gaps that exercise the narrow path, the 64-bit path
and the dropping rule, the float head bit for bit, and the error it hands back."""
import numpy as np
import pytest
import torch

import oracle
from oracle import ConvDesc
from paper_2105_13890_b200 import eoq, synth

import gpu_util as G

pytestmark = pytest.mark.gpu


def i32(v):
    return G.dev(np.array([v], dtype=np.int32))


POOLS = [  # n, h, w, c, k, stride, pad
    (2, 12, 12, 16, 3, 2, 1),      # the ImageNet networks' pool
    (3, 13, 11, 32, 3, 2, 1),      # odd sizes: the last window hangs over the border
    (2, 8, 8, 48, 2, 2, 0),        # disjoint windows
    (2, 9, 10, 16, 3, 1, 1),       # every position in nine windows
    (1, 7, 7, 16, 5, 3, 2),
    (5, 37, 41, 64, 3, 2, 1),      # several blocks, ragged tail
]


@pytest.mark.parametrize("n,h,w,c,k,s,p", POOLS)
@pytest.mark.parametrize("ties", [False, True])
def test_maxpool_forward_and_backward(n, h, w, c, k, s, p, ties):
    hd = G.handle()
    x = synth.relu_codes((n, h, w, c), 8100 + h, 0)
    if ties:
        x = (x // 32 * 32).astype(np.int8)      # few distinct values: most windows hold their maximum several times
    y_o, idx = oracle.maxpool_fwd(x, k, s, p)
    ho, wo = y_o.shape[1:3]
    e = synth.normal_codes((n, ho, wo, c), 8100 + h, 1)
    y, arg = G.zeros(y_o.shape, torch.int8), G.zeros(y_o.shape, torch.uint8)
    eoq.eoq_aux_maxpool_fwd(hd, G.dev(x), n, h, w, c, k, s, p, y, arg)
    ein, pin = G.zeros(x.shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_aux_maxpool_bwd(hd, G.dev(e), i32(-12), arg, n, h, w, c, k, s, p, ein, pin)
    torch.cuda.synchronize()
    assert np.array_equal(G.host(y), y_o)
    # the recorded position is the oracle's first maximum
    a = G.host(arg).astype(np.int64)
    b_, oy, ox, ch = np.meshgrid(np.arange(n), np.arange(ho), np.arange(wo), np.arange(c), indexing="ij")
    flat = ((b_ * h + (oy * s - p + a // k)) * w + (ox * s - p + a % k)) * c + ch
    assert np.array_equal(flat, idx)
    S = oracle.maxpool_bwd(e, idx, x.shape)
    codes, p_out, _ = oracle.sq_int(S, -12)
    assert np.array_equal(G.host(ein), codes) and pin.item() == p_out
    assert eoq.eoq_last_status(hd) == 0


@pytest.mark.parametrize("n,h,w,c,k,s,p", POOLS[:4] + POOLS[5:])
@pytest.mark.parametrize("gamma", [128, 37, -300])
def test_maxpool_backward_with_the_error_head_fused(n, h, w, c, k, s, p, gamma):
    """eoq_aux_maxpool_bwd_head against the oracle's pool backward followed by its error head, and against the two
    separate GPU calls; with and without the intermediate error written."""
    hd = G.handle()
    x = synth.relu_codes((n, h, w, c), 8150 + h, 0)
    _, idx = oracle.maxpool_fwd(x, k, s, p)
    ho, wo = idx.shape[1:3]
    e = synth.normal_codes((n, ho, wo, c), 8150 + h, 1)
    mask01 = synth.bits((n, h, w, c), 8150 + h, 2, 0.55)
    S = oracle.maxpool_bwd(e, idx, x.shape)
    e0, p0, _ = oracle.sq_int(S, -12)
    want_e3, want_p3, want_s1, _, _ = oracle.err_prescale(e0.astype(np.int8), p0, mask01, None, gamma)
    y, arg = G.zeros((n, ho, wo, c), torch.int8), G.zeros((n, ho, wo, c), torch.uint8)
    eoq.eoq_aux_maxpool_fwd(hd, G.dev(x), n, h, w, c, k, s, p, y, arg)
    g_d = i32(gamma)
    for keep in (True, False):
        ein, pin = G.zeros(x.shape, torch.int8), G.zeros(1, torch.int32)
        e3, p3, s1 = G.zeros(x.shape, torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
        eoq.eoq_aux_maxpool_bwd_head(hd, G.dev(e), i32(-12), arg, n, h, w, c, k, s, p, ein if keep else None, pin, G.dev(G.pack_mask(mask01)),
                                     g_d, e3, p3, s1)
        torch.cuda.synchronize()
        assert eoq.eoq_last_status(hd) == 0
        if keep:
            assert np.array_equal(G.host(ein), e0)
        assert pin.item() == p0
        assert np.array_equal(G.host(e3), want_e3) and p3.item() == want_p3 and s1.item() == want_s1


def test_maxpool_backward_of_a_zero_error_keeps_the_exponent():
    hd = G.handle()
    n, h, w, c = 1, 6, 6, 16
    x = synth.relu_codes((n, h, w, c), 8200, 0)
    y, arg = G.zeros((n, 3, 3, c), torch.int8), G.zeros((n, 3, 3, c), torch.uint8)
    eoq.eoq_aux_maxpool_fwd(hd, G.dev(x), n, h, w, c, 3, 2, 1, y, arg)
    ein, pin = G.empty((n, h, w, c), torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_aux_maxpool_bwd(hd, G.zeros((n, 3, 3, c), torch.int8), i32(-9), arg, n, h, w, c, 3, 2, 1, ein, pin)
    torch.cuda.synchronize()
    assert not G.host(ein).any() and pin.item() == -9
    assert eoq.eoq_last_status(hd) == eoq.EOQ_DEV_SQ_ZERO
    G.status_clear()


@pytest.mark.parametrize("n,hw,c", [(2, 49, 512), (3, 64, 64), (1, 1, 16), (4, 300, 32)])
def test_avgpool_sum(n, hw, c):
    hd = G.handle()
    x = synth.relu_codes((n, hw, 1, c), 8300 + hw, 0)
    sums = G.zeros((n, c), torch.int32)
    eoq.eoq_aux_avgpool_sum(hd, G.dev(x), n, hw, c, sums)
    torch.cuda.synchronize()
    assert np.array_equal(G.host(sums).astype(np.int64), oracle.avgpool_sum(x))


@pytest.mark.parametrize("pa,pb", [(-12, -12), (-11, -14), (-14, -11), (-10, -33), (-5, -40), (-40, -5), (-20, -51), (-52, -20)])
@pytest.mark.parametrize("gated", [False, True])
def test_join(pa, pb, gated):
    """Equal exponents, small gaps (32-bit path), gaps above 23 octaves (64-bit path) and above 31 (the smaller
    operand is dropped), with and without the gate bits of operand b."""
    hd = G.handle()
    shape = (3, 9, 7, 48)                      # 9072 codes: whole 16-code groups, several blocks, a ragged tail
    a = synth.normal_codes(shape, 8400, 0)
    b = synth.normal_codes(shape, 8400, 1)
    mask01 = (synth.relu_codes(shape, 8400, 2) > 0).astype(np.uint8) if gated else None
    S, p = oracle.join(a, pa, b, pb, mask01)
    codes, p_out, _ = oracle.sq_int(S, p)
    out, pout, ssum = G.zeros(shape, torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
    eoq.eoq_aux_join(hd, G.dev(a), i32(pa), G.dev(b), i32(pb), G.dev(G.pack_mask(mask01)) if gated else None, a.size, out, pout, ssum)
    torch.cuda.synchronize()
    assert np.array_equal(G.host(out), codes) and pout.item() == p_out
    assert ssum.item() == int(codes.astype(np.int64).sum())
    assert eoq.eoq_last_status(hd) == 0


@pytest.mark.parametrize("pa,pb", [(-12, -12), (-11, -14), (-10, -36), (-40, -5)])
@pytest.mark.parametrize("gamma,with_x2", [(118, True), (128, False), (-77, True)])
def test_join_with_the_consumer_error_head_fused(pa, pb, gamma, with_x2):
    """eoq_aux_join_head against the oracle's join followed by its error head (both 32- and 64-bit paths of the join)."""
    hd = G.handle()
    shape = (3, 9, 7, 48)
    a = synth.normal_codes(shape, 8450, 0)
    b = synth.normal_codes(shape, 8450, 1)
    gate01 = (synth.relu_codes(shape, 8450, 2) > 0).astype(np.uint8)
    mask01 = synth.bits(shape, 8450, 3, 0.5)
    x2 = (synth.relu_codes(shape, 8450, 4).astype(np.int32) * 37 - 900).astype(np.int16) if with_x2 else None
    S, p = oracle.join(a, pa, b, pb, gate01)
    codes, p_out, _ = oracle.sq_int(S, p)
    want_e3, want_p3, want_s1, want_s2, _ = oracle.err_prescale(codes.astype(np.int8), p_out, mask01, x2, gamma)
    out, pout, ssum = G.zeros(shape, torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
    e3, p3 = G.zeros(shape, torch.int8), G.zeros(1, torch.int32)
    s1, s2 = G.zeros(1, torch.int64), G.zeros(1, torch.int64)
    eoq.eoq_aux_join_head(hd, G.dev(a), i32(pa), G.dev(b), i32(pb), G.dev(G.pack_mask(gate01)), a.size, out, pout, ssum,
                          G.dev(G.pack_mask(mask01)), G.dev(x2) if with_x2 else None, i32(gamma), e3, p3, s1, s2 if with_x2 else None)
    torch.cuda.synchronize()
    assert eoq.eoq_last_status(hd) == 0
    assert np.array_equal(G.host(out), codes) and pout.item() == p_out and ssum.item() == int(codes.astype(np.int64).sum())
    assert np.array_equal(G.host(e3), want_e3) and p3.item() == want_p3 and s1.item() == want_s1
    if with_x2:
        assert s2.item() == want_s2
    # the handle's cells are clean again: a plain join right after gives the plain result
    out2, pout2 = G.zeros(shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_aux_join(hd, G.dev(a), i32(pa), G.dev(b), i32(pb), G.dev(G.pack_mask(gate01)), a.size, out2, pout2, None)
    torch.cuda.synchronize()
    assert np.array_equal(G.host(out2), codes) and pout2.item() == p_out


@pytest.mark.parametrize("n,c,hw,classes", [(2, 64, 64, 10), (5, 512, 49, 1000), (33, 64, 64, 10), (64, 512, 49, 1000)])
def test_float_head_bit_for_bit(n, c, hw, classes):
    hd = G.handle()
    sums = (synth.relu_codes((n, c), 8500 + n, 0).astype(np.int64) * hw) // 3
    W = (synth.normal_f32((classes, c), 8500 + n, 1) / np.float32(np.sqrt(c))).astype(np.float32)
    bias = (synth.normal_f32((classes,), 8500 + n, 2) * np.float32(0.01)).astype(np.float32)
    labels = synth.labels(n, classes, 8500 + n, 3).astype(np.int32)
    W_o, bias_o = W.copy(), bias.copy()
    loss_o, dpooled_o, logits_o = oracle.head(sums, hw, W_o, bias_o, labels, 2.0 ** -6)
    W_d, bias_d = G.dev(W), G.dev(bias)
    loss, dpooled, logits = G.zeros(1, torch.float32), G.zeros((n, c), torch.float32), G.zeros((n, classes), torch.float32)
    ws = G.zeros(eoq.eoq_aux_head_workspace_size(n, c, classes), torch.uint8)
    eoq.eoq_aux_head(hd, G.dev(sums.astype(np.int32)), n, c, hw, classes, W_d, bias_d, G.dev(labels), 2.0 ** -6, loss, dpooled, logits, ws)
    e, pe = G.zeros((n, hw, 1, c), torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_aux_head_error(hd, dpooled, n, c, hw, e, pe, ws)
    torch.cuda.synchronize()
    assert np.array_equal(G.host(logits), logits_o)
    assert np.array_equal(G.host(dpooled), dpooled_o)
    assert np.array_equal(G.host(W_d), W_o) and np.array_equal(G.host(bias_d), bias_o)
    assert loss.item() == pytest.approx(loss_o, rel=1e-6)
    # the SGD step taken apart from the rest gives the same parameters
    W2, bias2 = G.dev(W), G.dev(bias)
    eoq.eoq_aux_head(hd, G.dev(sums.astype(np.int32)), n, c, hw, classes, W2, bias2, G.dev(labels), 0.0, loss, dpooled, logits, ws)
    torch.cuda.synchronize()
    assert np.array_equal(G.host(W2), W) and np.array_equal(G.host(bias2), bias) and np.array_equal(G.host(dpooled), dpooled_o)
    eoq.eoq_aux_head_update(hd, n, c, classes, W2, bias2, 2.0 ** -6, ws)
    torch.cuda.synchronize()
    assert np.array_equal(G.host(W2), W_o) and np.array_equal(G.host(bias2), bias_o)
    # the error handed back: SQ of dpooled / hw, the same code at every position of a (sample, channel)
    codes, p_e, _ = oracle.quantize_f32(oracle.MODE_SQ, (dpooled_o / np.float32(hw)).astype(np.float32))
    got = G.host(e).reshape(n, hw, c)
    assert pe.item() == p_e and all(np.array_equal(got[:, i, :], codes) for i in (0, hw // 2, hw - 1))
    assert eoq.eoq_last_status(hd) == 0


DGRADS = [  # n, h, w, c_in, c_out, k, stride, pad
    (2, 12, 12, 32, 32, 3, 1, 1),      # patch kernel
    (3, 7, 7, 64, 128, 3, 1, 1),       # small image: per-tap kernel
    (2, 10, 10, 32, 64, 3, 2, 1),      # strided: four residue classes side by side
    (2, 9, 11, 48, 32, 1, 1, 0),       # 1x1
    (1, 20, 20, 64, 64, 5, 1, 2),
]


@pytest.mark.parametrize("n,h,w,c_in,c_out,k,stride,pad", DGRADS)
@pytest.mark.parametrize("gamma,with_x2", [(128, False), (91, True)])
def test_dgrad_with_the_consumer_error_head_fused(n, h, w, c_in, c_out, k, stride, pad, gamma, with_x2):
    """eoq_conv_dgrad_head against the oracle's dgrad + Q_e followed by its error head."""
    hd = G.handle()
    d = ConvDesc(n, h, w, c_in, c_out, k, k, stride, pad)
    gd = G.gdesc(d)
    e3 = synth.normal_codes((n, d.ho, d.wo, c_out), 8600 + h, 0)
    wt = synth.int8_uniform((c_out, k, k, c_in), 8600 + h, 1, -30, 30)
    in_shape = (n, h, w, c_in)
    mask01 = synth.bits(in_shape, 8600 + h, 2, 0.5)
    x2 = (synth.relu_codes(in_shape, 8600 + h, 3).astype(np.int32) * 29 - 700).astype(np.int16) if with_x2 else None
    S = oracle.conv_dgrad_acc(d, e3, wt)
    e4_o, p4_o, _ = oracle.sq_int(S, -11 - 7)
    want_e3, want_p3, want_s1, want_s2, _ = oracle.err_prescale(e4_o.astype(np.int8), p4_o, mask01, x2, gamma)
    e4, p4, s4 = G.zeros(in_shape, torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
    n3, pn3 = G.zeros(in_shape, torch.int8), G.zeros(1, torch.int32)
    s1, s2 = G.zeros(1, torch.int64), G.zeros(1, torch.int64)
    eoq.eoq_conv_dgrad_head(hd, gd, G.dev(e3), i32(-11), G.dev(wt), e4, p4, s4, G.dev(G.pack_mask(mask01)),
                            G.dev(x2) if with_x2 else None, i32(gamma), n3, pn3, s1, s2 if with_x2 else None,
                            G.workspace(gd, eoq.EOQ_PASS_DGRAD))
    torch.cuda.synchronize()
    assert eoq.eoq_last_status(hd) == 0
    assert np.array_equal(G.host(e4), e4_o) and p4.item() == p4_o and s4.item() == int(e4_o.astype(np.int64).sum())
    assert np.array_equal(G.host(n3), want_e3) and pn3.item() == want_p3 and s1.item() == want_s1
    if with_x2:
        assert s2.item() == want_s2
    # the plain call right after finds clean cells
    e4b, p4b = G.zeros(in_shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_conv_dgrad(hd, gd, G.dev(e3), i32(-11), G.dev(wt), e4b, p4b, None, None, G.workspace(gd, eoq.EOQ_PASS_DGRAD))
    torch.cuda.synchronize()
    assert np.array_equal(G.host(e4b), e4_o) and p4b.item() == p4_o


def test_dgrad_head_refuses_the_compact_strided_1x1_case():
    hd = G.handle()
    d = ConvDesc(2, 8, 8, 32, 64, 1, 1, 2, 0)
    gd = G.gdesc(d)
    z8 = lambda shape: G.zeros(shape, torch.int8)
    with pytest.raises(eoq.EoqError):
        eoq.eoq_conv_dgrad_head(hd, gd, z8((2, 4, 4, 64)), i32(-11), z8((64, 1, 1, 32)), z8((2, 8, 8, 32)), G.zeros(1, torch.int32), None,
                                G.zeros(2 * 8 * 8 * 32 // 8, torch.uint8), None, i32(128), z8((2, 8, 8, 32)), G.zeros(1, torch.int32),
                                None, None, G.workspace(gd, eoq.EOQ_PASS_DGRAD))


@pytest.mark.parametrize("n,h,w,c_in,c_out,k,stride,pad", DGRADS)
@pytest.mark.parametrize("pb,gated,with_head", [(-17, True, True), (-20, False, True), (-50, True, False), (-3, True, True)])
def test_dgrad_join_and_head_in_one_call(n, h, w, c_in, c_out, k, stride, pad, pb, gated, with_head):
    """eoq_conv_dgrad_join_head against the oracle's dgrad + Q_e, join + Q_e and error head (join exponents that take the
    32-bit path, the 64-bit path and the dropping rule in both directions)."""
    hd = G.handle()
    d = ConvDesc(n, h, w, c_in, c_out, k, k, stride, pad)
    gd = G.gdesc(d)
    e3 = synth.normal_codes((n, d.ho, d.wo, c_out), 8650 + h, 0)
    wt = synth.int8_uniform((c_out, k, k, c_in), 8650 + h, 1, -30, 30)
    in_shape = (n, h, w, c_in)
    b = synth.normal_codes(in_shape, 8650 + h, 2)
    gate01 = synth.bits(in_shape, 8650 + h, 3, 0.6) if gated else None
    mask01 = synth.bits(in_shape, 8650 + h, 4, 0.5)
    x2 = (synth.relu_codes(in_shape, 8650 + h, 5).astype(np.int32) * 23 - 500).astype(np.int16)
    S = oracle.conv_dgrad_acc(d, e3, wt)
    e4_o, p4_o, _ = oracle.sq_int(S, -11 - 7)
    J, pj = oracle.join(e4_o.astype(np.int8), p4_o, b, pb, gate01)
    out_o, pout_o, _ = oracle.sq_int(J, pj)
    want_e3, want_p3, want_s1, want_s2, _ = oracle.err_prescale(out_o.astype(np.int8), pout_o, mask01, x2, 97)
    e4, p4, s4 = G.zeros(in_shape, torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
    out, pout, sout = G.zeros(in_shape, torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
    n3, pn3 = G.zeros(in_shape, torch.int8), G.zeros(1, torch.int32)
    s1, s2 = G.zeros(1, torch.int64), G.zeros(1, torch.int64)
    head = (G.dev(G.pack_mask(mask01)), G.dev(x2), i32(97), n3, pn3, s1, s2) if with_head else (None,) * 7
    eoq.eoq_conv_dgrad_join_head(hd, gd, G.dev(e3), i32(-11), G.dev(wt), e4, p4, s4, G.dev(b), i32(pb),
                                 G.dev(G.pack_mask(gate01)) if gated else None, out, pout, sout, *head,
                                 workspace=G.workspace(gd, eoq.EOQ_PASS_DGRAD))
    torch.cuda.synchronize()
    assert eoq.eoq_last_status(hd) == 0
    assert np.array_equal(G.host(e4), e4_o) and p4.item() == p4_o and s4.item() == int(e4_o.astype(np.int64).sum())
    assert np.array_equal(G.host(out), out_o) and pout.item() == pout_o and sout.item() == int(out_o.astype(np.int64).sum())
    if with_head:
        assert np.array_equal(G.host(n3), want_e3) and pn3.item() == want_p3 and s1.item() == want_s1 and s2.item() == want_s2
    # every cell of the handle is clean again: the plain calls give the plain results
    e4b, p4b = G.zeros(in_shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_conv_dgrad(hd, gd, G.dev(e3), i32(-11), G.dev(wt), e4b, p4b, None, None, G.workspace(gd, eoq.EOQ_PASS_DGRAD))
    out2, pout2 = G.zeros(in_shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_aux_join(hd, e4b, p4b, G.dev(b), i32(pb), G.dev(G.pack_mask(gate01)) if gated else None, b.size, out2, pout2, None)
    torch.cuda.synchronize()
    assert np.array_equal(G.host(out2), out_o) and pout2.item() == pout_o

"""GPU parity: every C-ABI entry point against the oracle, element by element, on seeded synthetic inputs.
Integer tensors must match bit for bit; exponents are integers and must be equal."""
import numpy as np
import pytest
import torch

import oracle
from oracle import ConvDesc
from paper_2105_13890_b200 import eoq, synth

import gpu_util as G

pytestmark = pytest.mark.gpu

# geometry sweep: several tiles, ragged tails, every swizzle width, strides, 1x1 and 7x7, tiny images
SHAPES = [
    ConvDesc(8, 32, 32, 16, 16, 3, 3, 1, 1),      # the single-layer configuration
    ConvDesc(2, 8, 8, 64, 64, 3, 3, 1, 1),
    ConvDesc(3, 13, 11, 32, 48, 3, 3, 1, 1),      # ragged last tile, 48 columns
    ConvDesc(2, 10, 10, 128, 128, 3, 3, 1, 1),
    ConvDesc(1, 14, 14, 256, 512, 3, 3, 1, 1),    # two column tiles
    ConvDesc(3, 9, 7, 64, 48, 3, 3, 2, 1),        # stride 2, odd extents
    ConvDesc(2, 16, 16, 64, 128, 3, 3, 2, 1),
    ConvDesc(2, 8, 8, 64, 128, 1, 1, 1, 0),
    ConvDesc(2, 16, 16, 64, 128, 1, 1, 2, 0),     # projection shortcut
    ConvDesc(2, 20, 20, 16, 64, 7, 7, 2, 3),      # stem-like
    ConvDesc(1, 2, 2, 16, 16, 3, 3, 1, 1),        # every pixel touches the border
    ConvDesc(1, 1, 1, 32, 16, 1, 1, 1, 0),        # degenerate: one pixel
    ConvDesc(5, 7, 7, 512, 512, 3, 3, 1, 1),      # K = 4608
    ConvDesc(2, 12, 12, 192, 80, 3, 3, 1, 1),     # channel counts that are not powers of two
]
IDS = [f"n{d.n}_{d.h}x{d.w}_c{d.c_in}-{d.c_out}_k{d.kh}s{d.stride}p{d.pad}" for d in SHAPES]


def layer_data(d, seed, wrange=30):
    x0 = synth.relu_codes((d.n, d.h, d.w, d.c_in), seed, 0) if seed % 2 else synth.int8_uniform((d.n, d.h, d.w, d.c_in), seed, 0)
    w = synth.int8_uniform((d.c_out, d.kh, d.kw, d.c_in), seed, 1, -wrange, wrange)
    sc = synth.int8_uniform((d.n, d.ho, d.wo, d.c_out), seed, 2)
    e3 = synth.normal_codes((d.n, d.ho, d.wo, d.c_out), seed, 3)
    return x0, w, sc, e3


@pytest.mark.parametrize("d", SHAPES, ids=IDS)
@pytest.mark.parametrize("scal", [(0, 128, 0, False, True), (-3, 90, 5, True, True), (7, -200, -40, True, False)],
                         ids=["init", "b1neg_sc", "b1pos_norelu"])
def test_conv_fwd(d, scal):
    b1, gamma, b2, use_sc, relu = scal
    x0, w, sc, _ = layer_data(d, 100 + d.c_in + d.h)
    ref = oracle.layer_forward(d, x0, b1, w, gamma, b2, sc if use_sc else None, relu)
    gd = G.gdesc(d)
    shape = ref["x5"].shape
    x5, x2, acc = G.zeros(shape, torch.int8), G.zeros(shape, torch.int16), G.zeros(shape, torch.int32)
    mask = G.zeros((ref["x5"].size + 7) // 8, torch.uint8)
    eoq.eoq_conv_fwd(G.handle(), gd, G.dev(x0), None, b1, G.dev(w), gamma, b2, G.dev(sc) if use_sc else None, relu,
                     x5, x2, mask, acc, G.workspace(gd, eoq.EOQ_PASS_FWD))
    assert G.status_clear() == 0
    assert np.array_equal(G.host(acc).astype(np.int64), ref["acc"])
    assert np.array_equal(G.host(x2).astype(np.int32), ref["x2"])
    assert np.array_equal(G.host(x5), ref["x5"])
    assert np.array_equal(G.unpack_mask(mask, shape), ref["mask"])


EXTREME_CASES = [
    (ConvDesc(2, 6, 6, 512, 32, 3, 3, 1, 1), (-127, 127, 64, -64, 0, 1), (-127, 127, 1, 2, 0, -1)),   # x2 saturates both ways
    (ConvDesc(2, 9, 9, 16, 32, 1, 1, 1, 0), (0, 64, -64, 127), (0, 64, -64, 1)),                        # ties of both roundings
    (ConvDesc(2, 9, 9, 16, 32, 3, 3, 1, 1), (0, 64, -64), (0, 64, -64, 32)),
    (ConvDesc(1, 8, 8, 64, 64, 3, 3, 2, 1), (0, 64, -64, 1, -1), (0, 64, -64, 127, -127)),
]


@pytest.mark.parametrize("case", EXTREME_CASES, ids=["saturate", "ties_1x1", "ties_3x3", "ties_s2"])
@pytest.mark.parametrize("scal", [(0, 1, 0, False, True), (0, 1, 0, True, False), (5, 32767, -300, True, True),
                                  (-5, -32768, 300, True, False), (0, 127, 1, False, False), (0, -1, 0, False, True)],
                         ids=["g1", "g1_sc_norelu", "gmax", "gmin_norelu", "g127_norelu", "gneg1"])
def test_conv_fwd_ties_and_saturation(case, scal):
    """Operands drawn from a few extreme values: accumulators sit on rounding ties and beyond the 16-bit range
    of x2, and x4 reaches both ends of its range, so every clamp and tie of the forward chain is exercised."""
    d, xvals, wvals = case
    b1, gamma, b2, use_sc, relu = scal
    rng = np.random.Generator(np.random.Philox(key=[d.c_in, d.kh]))
    x0 = rng.choice(np.array(xvals, dtype=np.int8), size=(d.n, d.h, d.w, d.c_in))
    w = rng.choice(np.array(wvals, dtype=np.int8), size=(d.c_out, d.kh, d.kw, d.c_in))
    if case is EXTREME_CASES[0]:  # coherent signs: half of the output channels sum far up, a quarter far down
        x0 = np.abs(x0)
        w[0::2] = np.abs(w[0::2])
        w[1::4] = -np.abs(w[1::4])
    sc = rng.choice(np.array([-127, -1, 0, 1, 127], dtype=np.int8), size=(d.n, d.ho, d.wo, d.c_out))
    ref = oracle.layer_forward(d, x0, b1, w, gamma, b2, sc if use_sc else None, relu)
    gd = G.gdesc(d)
    shape = ref["x5"].shape
    x5, x2, acc = G.zeros(shape, torch.int8), G.zeros(shape, torch.int16), G.zeros(shape, torch.int32)
    mask = G.zeros((ref["x5"].size + 7) // 8, torch.uint8)
    eoq.eoq_conv_fwd(G.handle(), gd, G.dev(x0), None, b1, G.dev(w), gamma, b2, G.dev(sc) if use_sc else None, relu,
                     x5, x2, mask, acc, G.workspace(gd, eoq.EOQ_PASS_FWD))
    assert G.status_clear() == 0
    assert np.array_equal(G.host(acc).astype(np.int64), ref["acc"])
    assert np.array_equal(G.host(x2).astype(np.int32), ref["x2"])
    assert np.array_equal(G.host(x5), ref["x5"])
    assert np.array_equal(G.unpack_mask(mask, shape), ref["mask"])
    if case is EXTREME_CASES[0]:
        assert ref["x2"].max() == 32767 and ref["x2"].min() == -32768
    if case is EXTREME_CASES[1] and b1 == 0:
        assert np.any(np.abs(ref["acc"]) % 128 == 64)


MARGIN_CASES = [
    (ConvDesc(2, 20, 20, 16, 64, 7, 7, 2, 3), 4),     # filter-row path of the 7x7 stride-2 first layer
    (ConvDesc(3, 17, 23, 16, 32, 7, 7, 2, 3), 5),     # odd extents, wider margin
    (ConvDesc(2, 12, 12, 16, 16, 5, 5, 1, 2), 4),     # 5 taps wide, stride 1
    (ConvDesc(2, 20, 20, 16, 64, 7, 7, 2, 3), 2),     # margin too small for the filter-row path: per-tap path
    (ConvDesc(2, 9, 9, 32, 48, 3, 3, 1, 1), 3),       # margins on an ordinary layer
    (ConvDesc(2, 20, 20, 8, 64, 7, 7, 2, 3), 5),      # 8-channel input: a filter row is a 64-byte K slice
    (ConvDesc(3, 18, 22, 8, 32, 7, 7, 2, 3), 7),      # 8 channels, unequal extents, wider margin
    (ConvDesc(2, 16, 16, 8, 16, 5, 5, 2, 2), 4),      # 8 channels, 5 taps, pad 2
]


def with_margin(x0, m):
    return np.pad(x0, ((0, 0), (0, 0), (m, m), (0, 0)))


@pytest.mark.parametrize("d,m", MARGIN_CASES, ids=[f"k{d.kh}s{d.stride}_c{d.c_in}_m{m}_{d.h}x{d.w}" for d, m in MARGIN_CASES])
def test_input_with_row_margins(d, m):
    """Forward and weight gradient on an input stored with zero row margins (x_wmargin)."""
    x0, w, _, e3 = layer_data(d, 900 + m + d.h)
    gd = eoq.conv_desc(d.n, d.h, d.w, d.c_in, d.c_out, d.kh, d.kw, d.stride, d.pad, m)
    xm = G.dev(with_margin(x0, m))
    for b1 in (0, -4):
        ref = oracle.layer_forward(d, x0, b1, w, 100, 2)
        shape = ref["x5"].shape
        x5, acc = G.zeros(shape, torch.int8), G.zeros(shape, torch.int32)
        eoq.eoq_conv_fwd(G.handle(), gd, xm, None, b1, G.dev(w), 100, 2, None, True, x5, None, None, acc,
                         G.workspace(gd, eoq.EOQ_PASS_FWD))
        assert G.status_clear() == 0
        assert np.array_equal(G.host(acc).astype(np.int64), ref["acc"]) and np.array_equal(G.host(x5), ref["x5"])
        Gacc = oracle.conv_wgrad_acc(d, e3, x0, b1)
        g, pg, _ = oracle.sq_int(Gacc, -16)
        g_d, gacc, g_exp = G.zeros(Gacc.shape, torch.int8), G.zeros(Gacc.shape, torch.int64), G.zeros(1, torch.int32)
        eoq.eoq_conv_wgrad(G.handle(), gd, G.dev(e3), G.dev(np.array([-9], dtype=np.int32)), xm, b1, g_d, g_exp, gacc,
                           G.workspace(gd, eoq.EOQ_PASS_WGRAD))
        assert G.status_clear() == 0
        assert np.array_equal(G.host(gacc), Gacc) and g_exp.item() == pg
        assert np.array_equal(G.host(g_d).astype(np.int32), g)


@pytest.mark.parametrize("m,c_dst", [(0, 16), (4, 16), (5, 8), (0, 8)])
def test_quantize_image_pads_channels_and_rows(m, c_dst):
    n, h, w = 3, 10, 13
    img = synth.normal_f32((n, h, w, 3), 950, m)
    padded = np.zeros((n, h, w, c_dst), dtype=np.float32)
    padded[..., :3] = img
    c, p, _ = oracle.quantize_f32(oracle.MODE_SQ, padded)
    out = torch.full((n, h, w + 2 * m, c_dst), 55, dtype=torch.int8, device="cuda:0")
    ex = G.zeros(1, torch.int32)
    eoq.eoq_quantize_image(G.handle(), G.dev(img), n, h, w, 3, c_dst, m, out, ex)
    assert G.status_clear() == 0 and ex.item() == p
    assert np.array_equal(G.host(out).astype(np.int32), with_margin(c, m))


def test_conv_fwd_without_optional_outputs_and_with_input_exponent():
    d = ConvDesc(2, 12, 12, 16, 32, 3, 3, 1, 1)
    x0, w, _, _ = layer_data(d, 7)
    gd = G.gdesc(d)
    for p_in in (-5, -9, -7):
        ref = oracle.layer_forward(d, x0, 0, w, 128, 3, None, True, x_exp=p_in)
        x5 = G.zeros(ref["x5"].shape, torch.int8)
        eoq.eoq_conv_fwd(G.handle(), gd, G.dev(x0), G.dev(np.array([p_in], dtype=np.int32)), 0, G.dev(w), 128, 3, None,
                         True, x5)
        assert G.status_clear() == 0
        assert np.array_equal(G.host(x5), ref["x5"])


@pytest.mark.parametrize("d", SHAPES, ids=IDS)
def test_conv_dgrad(d):
    _, w, _, e3 = layer_data(d, 200 + d.c_out + d.w)
    p3 = -11
    B = oracle.conv_dgrad_acc(d, e3, w)
    e4, p4, z = oracle.sq_int(B, p3 - 7)
    gd = G.gdesc(d)
    e4_d, acc = G.zeros(B.shape, torch.int8), G.zeros(B.shape, torch.int32)
    e4_exp, s4 = G.zeros(1, torch.int32), G.zeros(1, torch.int64)
    eoq.eoq_conv_dgrad(G.handle(), gd, G.dev(e3), G.dev(np.array([p3], dtype=np.int32)), G.dev(w), e4_d, e4_exp, s4,
                       acc, G.workspace(gd, eoq.EOQ_PASS_DGRAD))
    assert G.status_clear() == (eoq.EOQ_DEV_SQ_ZERO if z else 0)
    assert np.array_equal(G.host(acc).astype(np.int64), B)
    assert e4_exp.item() == p4
    assert np.array_equal(G.host(e4_d).astype(np.int32), e4)
    assert s4.item() == int(e4.astype(np.int64).sum())
    # same call with the sums kept in the workspace
    e4_b, exp_b = G.zeros(B.shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_conv_dgrad(G.handle(), gd, G.dev(e3), G.dev(np.array([p3], dtype=np.int32)), G.dev(w), e4_b, exp_b, None,
                       None, G.workspace(gd, eoq.EOQ_PASS_DGRAD))
    G.status_clear()
    assert torch.equal(e4_b, e4_d) and exp_b.item() == p4


@pytest.mark.parametrize("d", SHAPES, ids=IDS)
@pytest.mark.parametrize("b1", [0, -5])
def test_conv_wgrad(d, b1):
    x0, _, _, e3 = layer_data(d, 300 + d.c_in + d.w)
    p3 = -9
    Gacc = oracle.conv_wgrad_acc(d, e3, x0, b1)
    g, pg, z = oracle.sq_int(Gacc, p3 - 7)
    gd = G.gdesc(d)
    g_d, acc = G.zeros(Gacc.shape, torch.int8), G.zeros(Gacc.shape, torch.int64)
    g_exp = G.zeros(1, torch.int32)
    eoq.eoq_conv_wgrad(G.handle(), gd, G.dev(e3), G.dev(np.array([p3], dtype=np.int32)), G.dev(x0), b1, g_d, g_exp, acc,
                       G.workspace(gd, eoq.EOQ_PASS_WGRAD))
    assert G.status_clear() == (eoq.EOQ_DEV_SQ_ZERO if z else 0)
    assert np.array_equal(G.host(acc), Gacc)
    assert g_exp.item() == pg
    assert np.array_equal(G.host(g_d).astype(np.int32), g)


def test_wgrad_long_reduction_needs_more_than_int32():
    """All-extreme operands over 2^17+ pixels overflow an int32 sum; the split-K partials must still be exact."""
    d = ConvDesc(9, 128, 128, 16, 16, 1, 1, 1, 0)
    x0 = np.full((d.n, d.h, d.w, d.c_in), 127, dtype=np.int8)
    e3 = np.full((d.n, d.ho, d.wo, d.c_out), -127, dtype=np.int8)
    gd = G.gdesc(d)
    acc, g_d, g_exp = G.zeros((16, 1, 1, 16), torch.int64), G.zeros((16, 1, 1, 16), torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_conv_wgrad(G.handle(), gd, G.dev(e3), G.dev(np.array([0], dtype=np.int32)), G.dev(x0), 0, g_d, g_exp, acc,
                       G.workspace(gd, eoq.EOQ_PASS_WGRAD))
    assert G.status_clear() == 0
    want = -127 * 127 * d.n * d.h * d.w
    assert abs(want) > 2**31
    assert (G.host(acc) == want).all()


@pytest.mark.parametrize("n", [1, 15, 16, 4099, 1 << 20])
@pytest.mark.parametrize("mode", [eoq.EOQ_Q, eoq.EOQ_CQ, eoq.EOQ_SQ])
def test_quantize_f32(n, mode):
    x = synth.normal_f32(n, 400 + n % 97, mode, std=2.5 if mode != eoq.EOQ_SQ else 1e-3)
    c, p, flag = oracle.quantize_f32(mode, x)
    if mode == eoq.EOQ_Q:
        c = np.clip(c, -32768, 32767)
    out = G.zeros(n, torch.int16 if mode == eoq.EOQ_Q else torch.int8)
    ex = G.zeros(1, torch.int32)
    eoq.eoq_quantize(G.handle(), mode, G.dev(x), True, None, n, out, ex)
    assert G.status_clear() == 0
    assert np.array_equal(G.host(out).astype(np.int32), c) and ex.item() == p


def test_quantize_edge_cases():
    h = G.handle()
    out, ex = G.zeros(64, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_quantize(h, eoq.EOQ_SQ, G.zeros(64, torch.float32), True, None, 64, out, ex)
    assert G.status_clear() == eoq.EOQ_DEV_SQ_ZERO and not out.any() and ex.item() == -7
    x = np.ones(64, dtype=np.float32)
    x[5] = np.inf
    eoq.eoq_quantize(h, eoq.EOQ_SQ, G.dev(x), True, None, 64, out, ex)
    assert G.status_clear() & eoq.EOQ_DEV_NONFINITE
    # ties, saturation and subnormal magnitudes
    x = np.array([0.5 / 128, 1.5 / 128, -2.5 / 128, 300.0, -300.0, 1e-45, 0.99609375, 1.0] * 2, dtype=np.float32)
    for mode in (eoq.EOQ_Q, eoq.EOQ_CQ):
        c, _, _ = oracle.quantize_f32(mode, x)
        o = G.zeros(16, torch.int16 if mode == eoq.EOQ_Q else torch.int8)
        eoq.eoq_quantize(h, mode, G.dev(x), True, None, 16, o, None)
        assert np.array_equal(G.host(o).astype(np.int32), np.clip(c, -32768, 32767))
    tiny = (synth.normal_f32(333, 9, 9) * 1e-41).astype(np.float32)
    c, p, _ = oracle.quantize_f32(eoq.EOQ_SQ, tiny)
    o = G.zeros(333, torch.int8)
    eoq.eoq_quantize(h, eoq.EOQ_SQ, G.dev(tiny), True, None, 333, o, ex)
    assert G.status_clear() == 0 and np.array_equal(G.host(o).astype(np.int32), c) and ex.item() == p


@pytest.mark.parametrize("n", [16, 1000, 1 << 18])
def test_quantize_int32_source(n):
    a = synth.rng(500, n).integers(-2**27, 2**27, size=n).astype(np.int32)
    c, p, _ = oracle.sq_int(a.astype(np.int64), -19)
    out, ex = G.zeros(n, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_quantize(G.handle(), eoq.EOQ_SQ, G.dev(a), False, G.dev(np.array([-19], dtype=np.int32)), n, out, ex)
    assert G.status_clear() == 0
    assert np.array_equal(G.host(out).astype(np.int32), c) and ex.item() == p


@pytest.mark.parametrize("n_el", [16, 4096 + 16, 1 << 19])
@pytest.mark.parametrize("gamma", [128, -77, 3])
def test_err_prescale(n_el, gamma):
    e0 = synth.normal_codes(n_el, 600, gamma & 0xff)
    mask = synth.bits(n_el, 601, 0)
    x2 = synth.rng(602, 0).integers(-3000, 3001, size=n_el).astype(np.int16)
    p0 = -13
    e3, p3, s1, s2, z = oracle.err_prescale(e0, p0, mask, x2.astype(np.int32), gamma)
    e3_d, e3_exp = G.zeros(n_el, torch.int8), G.zeros(1, torch.int32)
    s1_d, s2_d = G.zeros(1, torch.int64), G.zeros(1, torch.int64)
    eoq.eoq_err_prescale(G.handle(), G.dev(e0), G.dev(np.array([p0], dtype=np.int32)), G.dev(G.pack_mask(mask)),
                         G.dev(x2), n_el, gamma, e3_d, e3_exp, s1_d, s2_d)
    assert G.status_clear() == 0
    assert np.array_equal(G.host(e3_d), e3) and e3_exp.item() == p3
    assert s1_d.item() == s1 and s2_d.item() == s2


def test_err_prescale_two_kernel_path():
    """Tensors too large for the one-kernel error head (more than 6 groups of 16 codes per resident thread) take
    the reduce + apply pair; the first layer of the ImageNet networks at batch 64 is such a tensor."""
    n_el = 14_720_000  # 920,000 groups of 16: above the one-kernel capacity of a 148-SM device (909,312 groups)
    gamma = 118
    e0 = synth.normal_codes(n_el, 610, 1)
    mask = synth.bits(n_el, 611, 0)
    p0 = -12
    e3, p3, s1, _, _ = oracle.err_prescale(e0, p0, mask, None, gamma)
    e3_d, e3_exp, s1_d = G.zeros(n_el, torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
    h = G.handle()
    before = eoq.eoq_launch_count(h)
    for _ in range(2):  # twice: the reduction cells must come back clean
        eoq.eoq_err_prescale(h, G.dev(e0), G.dev(np.array([p0], dtype=np.int32)), G.dev(G.pack_mask(mask)), None, n_el,
                             gamma, e3_d, e3_exp, s1_d, None)
        assert G.status_clear() == 0
        assert np.array_equal(G.host(e3_d), e3) and e3_exp.item() == p3 and s1_d.item() == s1
    assert eoq.eoq_launch_count(h) - before == 4  # two kernels per call


@pytest.mark.parametrize("stochastic", [False, True])
def test_update_multi_tensor(stochastic):
    sizes = [16, 2304, 36864 + 5, 100000, 1, 8192, 8193]
    r = synth.rng(700, int(stochastic))
    ws = [synth.int8_uniform(n, 701, i) for i, n in enumerate(sizes)]
    gs = [synth.normal_codes(n, 702, i, std_codes=40) for i, n in enumerate(sizes)]
    pgs = [int(v) for v in r.integers(-16, -4, size=len(sizes))]
    gs[4][:] = 0  # an all-zero gradient leaves its tensor untouched
    for lr_mant, lr_exp in ((1, -3), (37, -8), (255, 2)):
        w_d = [G.dev(w) for w in ws]
        eoq.eoq_update(G.handle(), w_d, [G.dev(g) for g in gs], [G.dev(np.array([p], dtype=np.int32)) for p in pgs],
                       lr_mant, lr_exp, eoq.EOQ_ROUND_STOCHASTIC if stochastic else eoq.EOQ_ROUND_RNE, seed=11, step=3)
        assert G.status_clear() == eoq.EOQ_DEV_SQ_ZERO
        changed = 0
        for i, (w, g, p) in enumerate(zip(ws, gs, pgs)):
            want, _, _ = oracle.update(w, g, p, lr_mant, lr_exp, stochastic=stochastic, seed=11, step=3, tensor_id=i)
            got = G.host(w_d[i]).astype(np.int32)
            assert np.array_equal(got, want), (i, lr_mant, lr_exp)
            changed += int((got != w).sum())
        assert changed > 0


def test_layout_convert_round_trip():
    x = synth.int8_uniform((3, 20, 7, 9), 800, 0)  # NCHW
    nhwc, back = G.zeros((3, 7, 9, 20), torch.int8), G.zeros((3, 20, 7, 9), torch.int8)
    eoq.eoq_layout_convert(G.handle(), G.dev(x), nhwc, 3, 20, 7, 9, True)
    eoq.eoq_layout_convert(G.handle(), nhwc, back, 3, 20, 7, 9, False)
    assert np.array_equal(G.host(nhwc), x.transpose(0, 2, 3, 1)) and np.array_equal(G.host(back), x)


def test_argument_errors_launch_nothing():
    h = G.handle()
    d = eoq.conv_desc(1, 8, 8, 16, 16, 3, 3, 1, 1)
    x, w, y = G.zeros((1, 8, 8, 16), torch.int8), G.zeros((16, 3, 3, 16), torch.int8), G.zeros((1, 8, 8, 16), torch.int8)
    assert eoq.eoq_conv_fwd(h, eoq.conv_desc(1, 8, 8, 12, 16, 3, 3, 1, 1), x, None, 0, w, 128, 0, None, True, y, check=False) == eoq.EOQ_ERR_ALIGNMENT
    assert eoq.eoq_conv_fwd(h, d, x, None, 0, w, 1 << 20, 0, None, True, y, check=False) == eoq.EOQ_ERR_RANGE
    assert eoq.eoq_conv_fwd(h, d, x, None, 4, w, 128, 0, None, True, y, check=False) == eoq.EOQ_ERR_WORKSPACE
    assert eoq.eoq_conv_fwd(h, d, None, None, 0, w, 128, 0, None, True, y, check=False) == eoq.EOQ_ERR_BAD_ARG
    assert eoq.eoq_conv_fwd(h, d, x.data_ptr() + 1, None, 0, w, 128, 0, None, True, y, check=False) == eoq.EOQ_ERR_ALIGNMENT
    ex = G.zeros(1, torch.int32)
    assert eoq.eoq_conv_dgrad(h, d, y, ex, w, x, ex, check=False) == eoq.EOQ_ERR_WORKSPACE
    assert eoq.eoq_conv_fwd(h, eoq.conv_desc(1, 8, 8, 16, 16, 9, 9, 1, 4), x, None, 0, w, 128, 0, None, True, y, check=False) == eoq.EOQ_ERR_UNSUPPORTED
    # 8 input channels exist only on the filter-row path: ordinary layers, odd margin distances and dgrad refuse them
    ws = G.zeros(1 << 20, torch.uint8)
    assert eoq.eoq_conv_fwd(h, eoq.conv_desc(1, 8, 8, 8, 16, 3, 3, 1, 1), x, None, 0, w, 128, 0, None, True, y, None, None, None, ws, check=False) == eoq.EOQ_ERR_UNSUPPORTED
    assert eoq.eoq_conv_fwd(h, eoq.conv_desc(1, 8, 8, 8, 16, 7, 7, 2, 3, 4), x, None, 0, w, 128, 0, None, True, y, None, None, None, ws, check=False) == eoq.EOQ_ERR_UNSUPPORTED
    assert eoq.eoq_conv_dgrad(h, eoq.conv_desc(1, 8, 8, 8, 16, 7, 7, 2, 3, 5), y, ex, w, x, ex, None, None, ws, check=False) == eoq.EOQ_ERR_UNSUPPORTED
    assert G.status_clear() == 0


@pytest.mark.parametrize("ctas", [1, 37, 74])
def test_gemm_cta_cap_does_not_change_results(ctas):
    """eoq_set_gemm_ctas only changes how many persistent CTAs walk the tiles: every output stays bit-identical
    to the oracle."""
    d = ConvDesc(6, 14, 14, 64, 128, 3, 3, 1, 1)
    x0, w, sc, e3 = layer_data(d, 4100 + ctas)
    gd = G.gdesc(d)
    h = eoq.eoq_create(0)
    eoq.eoq_set_gemm_ctas(h, ctas)
    ref = oracle.layer_forward(d, x0, -3, w, 90, 5, sc, True)
    x5 = G.zeros(ref["x5"].shape, torch.int8)
    eoq.eoq_conv_fwd(h, gd, G.dev(x0), None, -3, G.dev(w), 90, 5, G.dev(sc), True, x5, None, None, None,
                     G.workspace(gd, eoq.EOQ_PASS_FWD))
    assert np.array_equal(G.host(x5), ref["x5"])
    B = oracle.conv_dgrad_acc(d, e3, w)
    e4_ref, p4, _ = oracle.sq_int(B, -9 - 7)
    e4, e4_exp = G.zeros(x0.shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_conv_dgrad(h, gd, G.dev(e3), G.dev(np.array([-9], dtype=np.int32)), G.dev(w), e4, e4_exp, None, None,
                       G.workspace(gd, eoq.EOQ_PASS_DGRAD))
    assert np.array_equal(G.host(e4).astype(np.int32), e4_ref) and e4_exp.item() == p4
    Gacc = oracle.conv_wgrad_acc(d, e3, x0, -3)
    g_ref, pg, _ = oracle.sq_int(Gacc, -9 - 7)
    g_d, g_exp = G.zeros(Gacc.shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_conv_wgrad(h, gd, G.dev(e3), G.dev(np.array([-9], dtype=np.int32)), G.dev(x0), -3, g_d, g_exp, None,
                       G.workspace(gd, eoq.EOQ_PASS_WGRAD))
    assert np.array_equal(G.host(g_d).astype(np.int32), g_ref) and g_exp.item() == pg
    assert eoq.eoq_last_status(h) == 0
    with pytest.raises(eoq.EoqError):
        eoq.eoq_set_gemm_ctas(h, -1)
    eoq.eoq_destroy(h)


@pytest.mark.parametrize("d", [ConvDesc(2, 16, 16, 64, 128, 1, 1, 2, 0), ConvDesc(3, 9, 7, 32, 48, 1, 1, 2, 0),
                               ConvDesc(2, 10, 10, 64, 64, 1, 1, 3, 0)],
                         ids=["s2_even", "s2_odd_extents", "s3"])
def test_strided_1x1_dgrad_without_sum_dump(d):
    """Without an int32 dump a strided 1x1 filter takes the compact path (sums only on the stride grid, Q_e
    scatters them): e4 must carry the oracle's codes on the grid and exact zeros elsewhere."""
    _, w, _, e3 = layer_data(d, 5200 + d.h)
    B = oracle.conv_dgrad_acc(d, e3, w)
    ref, p4, _ = oracle.sq_int(B, -10 - 7)
    gd = G.gdesc(d)
    e4 = torch.full((d.n, d.h, d.w, d.c_in), 77, dtype=torch.int8, device="cuda:0")
    e4_exp, s4 = G.zeros(1, torch.int32), G.zeros(1, torch.int64)
    for _ in range(2):  # twice: the reduction cells must come back clean
        eoq.eoq_conv_dgrad(G.handle(), gd, G.dev(e3), G.dev(np.array([-10], dtype=np.int32)), G.dev(w), e4, e4_exp, s4, None,
                           G.workspace(gd, eoq.EOQ_PASS_DGRAD))
        assert G.status_clear() == 0
        assert np.array_equal(G.host(e4).astype(np.int32), ref) and e4_exp.item() == p4
        assert s4.item() == int(ref.astype(np.int64).sum())


# ------------------------------------------------------------------ paths that only large problems take

WIDE_CASES = [
    # (geometry, pass, expected fragment of the plan): a 256-column tile needs at least twice as many tiles as SMs
    (ConvDesc(13, 56, 56, 64, 256, 1, 1, 1, 0), eoq.EOQ_PASS_FWD, "kernel=igemm tile_n=256"),
    (ConvDesc(13, 56, 56, 256, 64, 1, 1, 1, 0), eoq.EOQ_PASS_DGRAD, "kernel=igemm classes=1 tile_n=256"),
    (ConvDesc(148, 14, 14, 256, 256, 3, 3, 1, 1), eoq.EOQ_PASS_FWD, "kernel=igemm_patch tile_n=256 accumulators=1"),
    (ConvDesc(148, 14, 14, 256, 256, 3, 3, 1, 1), eoq.EOQ_PASS_DGRAD, "kernel=igemm_patch tile_n=256 accumulators=1"),
]


@pytest.mark.parametrize("d,pass_,plan", WIDE_CASES, ids=["igemm_fwd", "igemm_dgrad", "patch_fwd", "patch_dgrad"])
def test_256_column_tiles(d, pass_, plan):
    """Both implicit-GEMM kernels with 256-column tiles (one accumulator per tile), which only problems with at
    least 2 x SMs row tiles take; the plan report confirms the path before the results are compared."""
    gd = G.gdesc(d)
    assert plan in eoq.eoq_describe_plan(G.handle(), gd, pass_)
    x0, w, sc, e3 = layer_data(d, 7300 + d.c_in, wrange=12)
    if pass_ == eoq.EOQ_PASS_FWD:
        ref = oracle.layer_forward(d, x0, -3, w, 90, 5, sc, True)
        shape = ref["x5"].shape
        x5, x2, acc = G.zeros(shape, torch.int8), G.zeros(shape, torch.int16), G.zeros(shape, torch.int32)
        mask = G.zeros((ref["x5"].size + 7) // 8, torch.uint8)
        eoq.eoq_conv_fwd(G.handle(), gd, G.dev(x0), None, -3, G.dev(w), 90, 5, G.dev(sc), True, x5, x2, mask, acc,
                         G.workspace(gd, eoq.EOQ_PASS_FWD))
        assert G.status_clear() == 0
        assert np.array_equal(G.host(acc).astype(np.int64), ref["acc"])
        assert np.array_equal(G.host(x2).astype(np.int32), ref["x2"])
        assert np.array_equal(G.host(x5), ref["x5"])
        assert np.array_equal(G.unpack_mask(mask, shape), ref["mask"])
    else:
        B = oracle.conv_dgrad_acc(d, e3, w)
        e4, p4, _ = oracle.sq_int(B, -11 - 7)
        e4_d, acc = G.zeros(B.shape, torch.int8), G.zeros(B.shape, torch.int32)
        e4_exp, s4 = G.zeros(1, torch.int32), G.zeros(1, torch.int64)
        eoq.eoq_conv_dgrad(G.handle(), gd, G.dev(e3), G.dev(np.array([-11], dtype=np.int32)), G.dev(w), e4_d, e4_exp, s4, acc,
                           G.workspace(gd, eoq.EOQ_PASS_DGRAD))
        assert G.status_clear() == 0
        assert np.array_equal(G.host(acc).astype(np.int64), B) and e4_exp.item() == p4
        assert np.array_equal(G.host(e4_d).astype(np.int32), e4) and s4.item() == int(e4.astype(np.int64).sum())


# ------------------------------------------------------------------ device-resident scalars and prepared weights

DEV_SHAPES = [SHAPES[0], SHAPES[3], SHAPES[5], SHAPES[8], SHAPES[12]]


@pytest.mark.parametrize("d", DEV_SHAPES, ids=[IDS[SHAPES.index(d)] for d in DEV_SHAPES])
def test_device_scalar_entry_points(d):
    """eoq_weight_prep + eoq_conv_fwd_dev, eoq_err_prescale_dev and eoq_conv_wgrad_dev against the oracle, with the
    scalars rewritten in device memory between two calls (what a replayed graph sees)."""
    x0, w, sc, _ = layer_data(d, 8100 + d.c_out)
    e0 = synth.normal_codes((d.n, d.ho, d.wo, d.c_out), 8101, d.h)
    gd = G.gdesc(d)
    h = G.handle()
    prep = G.zeros(max(eoq.eoq_weight_prep_size(gd), 256), torch.uint8)
    w_d = G.dev(w)
    eoq.eoq_weight_prep(h, [gd], [w_d], [prep])
    scal = G.zeros(3, torch.int32)
    shape = (d.n, d.ho, d.wo, d.c_out)
    x5, x2 = G.zeros(shape, torch.int8), G.zeros(shape, torch.int16)
    mask = G.zeros((int(np.prod(shape)) + 7) // 8, torch.uint8)
    e3, e3_exp = G.zeros(shape, torch.int8), G.zeros(1, torch.int32)
    s1, s2 = G.zeros(1, torch.int64), G.zeros(1, torch.int64)
    g_d, g_exp = G.zeros(w.shape, torch.int8), G.zeros(1, torch.int32)
    ws = G.workspace(gd, eoq.EOQ_PASS_WGRAD)
    for b1, gamma, b2 in ((-3, 90, 5), (6, -131, -9), (0, 128, 0)):
        scal.copy_(torch.tensor([b1, gamma, b2], dtype=torch.int32))
        ref = oracle.layer_forward(d, x0, b1, w, gamma, b2, sc, True)
        eoq.eoq_conv_fwd_dev(h, gd, G.dev(x0), None, scal, w_d, prep, G.dev(sc), True, x5, x2, mask)
        assert G.status_clear() == 0
        assert np.array_equal(G.host(x5), ref["x5"]) and np.array_equal(G.host(x2).astype(np.int32), ref["x2"])
        assert np.array_equal(G.unpack_mask(mask, shape), ref["mask"])
        bwd = oracle.layer_backward(d, e0, -12, ref["mask"], ref["x2"], x0, b1, w, gamma)
        eoq.eoq_err_prescale_dev(h, G.dev(e0), G.dev(np.array([-12], dtype=np.int32)), mask, x2, e0.size, scal[1:2], e3, e3_exp,
                                 s1, s2)
        eoq.eoq_conv_wgrad_dev(h, gd, e3, e3_exp, G.dev(x0), scal[0:1], g_d, g_exp, ws)
        z = bwd["g_w_zero"]
        assert G.status_clear() == (eoq.EOQ_DEV_SQ_ZERO if z else 0)
        assert np.array_equal(G.host(e3), bwd["e3"]) and e3_exp.item() == bwd["p3"]
        assert s1.item() == bwd["sum_e1"] and s2.item() == bwd["sum_e1x2"]
        assert np.array_equal(G.host(g_d), bwd["g_w"]) and g_exp.item() == bwd["p_gw"]


def test_device_scalars_out_of_range_are_flagged():
    d = SHAPES[1]
    x0, w, _, _ = layer_data(d, 8200)
    gd = G.gdesc(d)
    prep = G.zeros(max(eoq.eoq_weight_prep_size(gd), 256), torch.uint8)
    eoq.eoq_weight_prep(G.handle(), [gd], [G.dev(w)], [prep])
    x5 = G.zeros((d.n, d.ho, d.wo, d.c_out), torch.int8)
    scal = G.dev(np.array([0, 1 << 20, 0], dtype=np.int32))
    eoq.eoq_conv_fwd_dev(G.handle(), gd, G.dev(x0), None, scal, G.dev(w), prep, None, True, x5)
    assert G.status_clear() == eoq.EOQ_DEV_RANGE
    # a bias without prepared weights cannot be applied: flagged, counted as zero
    scal = G.dev(np.array([5, 128, 0], dtype=np.int32))
    eoq.eoq_conv_fwd_dev(G.handle(), gd, G.dev(x0), None, scal, G.dev(w), None, None, True, x5)
    assert G.status_clear() == eoq.EOQ_DEV_RANGE
    ref = oracle.layer_forward(d, x0, 0, w, 128, 0)
    assert np.array_equal(G.host(x5), ref["x5"])


def test_update_with_device_step_counter():
    sizes = [4096, 36864 + 5, 16]
    ws = [synth.int8_uniform(n, 8301, i) for i, n in enumerate(sizes)]
    gs = [synth.normal_codes(n, 8302, i, std_codes=40) for i, n in enumerate(sizes)]
    pgs = [-9, -11, -8]
    w_d = [G.dev(w) for w in ws]
    step = G.dev(np.array([5], dtype=np.int64))
    cur = [w.astype(np.int32) for w in ws]
    for k in range(3):
        eoq.eoq_update_dev(G.handle(), w_d, [G.dev(g) for g in gs], [G.dev(np.array([p], dtype=np.int32)) for p in pgs],
                           37, -8, eoq.EOQ_ROUND_STOCHASTIC, 11, step)
        assert G.status_clear() == 0
        for i in range(len(sizes)):
            cur[i], _, _ = oracle.update(cur[i], gs[i], pgs[i], 37, -8, stochastic=True, seed=11, step=5 + k, tensor_id=i)
            assert np.array_equal(G.host(w_d[i]).astype(np.int32), cur[i]), (k, i)
    assert step.item() == 8


def test_wgrad_two_kernel_finish_path():
    """A weight tensor too large for the one-kernel slice sum + Q_g (more sums than a resident grid keeps in
    registers) takes the finalize + Q_g pair."""
    d = ConvDesc(1, 6, 6, 1024, 1024, 3, 3, 1, 1)   # 9.4 M weights
    x0, _, _, e3 = layer_data(d, 8400)
    Gacc = oracle.conv_wgrad_acc(d, e3, x0, -2)
    g, pg, _ = oracle.sq_int(Gacc, -9 - 7)
    gd = G.gdesc(d)
    g_d, g_exp = G.zeros(Gacc.shape, torch.int8), G.zeros(1, torch.int32)
    h = G.handle()
    for _ in range(2):
        before = eoq.eoq_launch_count(h)
        eoq.eoq_conv_wgrad(h, gd, G.dev(e3), G.dev(np.array([-9], dtype=np.int32)), G.dev(x0), -2, g_d, g_exp, None,
                           G.workspace(gd, eoq.EOQ_PASS_WGRAD))
        assert G.status_clear() == 0
        assert eoq.eoq_launch_count(h) - before == 4  # tap sums, GEMM, finalize, Q_g
        assert np.array_equal(G.host(g_d).astype(np.int32), g) and g_exp.item() == pg


# ------------------------------------------------------------------ a bounded wait that runs out

def test_wait_that_runs_out_reports_timeout_and_leaves_the_handle_usable():
    """The grid-wide wait of the one-kernel error head is made to run out (it waits for one block more than
    exists, with a short limit).  Nothing traps or hangs: the kernel returns, EOQ_DEV_TIMEOUT is reported, no output
    is written, the reduction cells are clean again, and the next call on the handle is bit-exact."""
    n_el = 1 << 16
    e0 = synth.normal_codes(n_el, 8500, 1)
    mask = synth.bits(n_el, 8501, 0)
    ref, p3, s1, _, _ = oracle.err_prescale(e0, -12, mask, None, 118)
    h = eoq.eoq_create(0)
    try:
        e3 = torch.full((n_el,), 55, dtype=torch.int8, device="cuda:0")
        e3_exp, s1_d = torch.full((1,), 1234, dtype=torch.int32, device="cuda:0"), G.zeros(1, torch.int64)
        args = (G.dev(e0), G.dev(np.array([-12], dtype=np.int32)), G.dev(G.pack_mask(mask)), None, n_el, 118, e3, e3_exp, s1_d, None)
        eoq.eoq_debug_force_wait_timeout(h)
        eoq.eoq_err_prescale(h, *args)
        assert eoq.eoq_last_status(h) == eoq.EOQ_DEV_TIMEOUT
        assert (G.host(e3) == 55).all() and e3_exp.item() == 1234      # nothing was written
        assert eoq.eoq_last_status(h) == 0                             # reported once, then clear
        for _ in range(2):
            eoq.eoq_err_prescale(h, *args)
            assert eoq.eoq_last_status(h) == 0
            assert np.array_equal(G.host(e3), ref) and e3_exp.item() == p3 and s1_d.item() == s1
    finally:
        eoq.eoq_destroy(h)


# ------------------------------------------------------------------ other update widths

@pytest.mark.parametrize("k_u,k_m", [(8, 8), (16, 16), (24, 24), (8, 24)])
@pytest.mark.parametrize("stochastic", [False, True])
def test_update_at_other_widths(k_u, k_m, stochastic):
    """Three consecutive updates with a k_u-bit update quantizer on a k_m-bit master copy: master codes and the 8-bit
    weights derived from them against the oracle; with 24-bit masters, sub-LSB updates accumulate."""
    sizes = [4096 + 7, 36864, 16]
    lim = 2 ** (k_m - 1) - 1
    r = synth.rng(8600, k_m)
    masters = [r.integers(-lim, lim + 1, size=n).astype(np.int32) for n in sizes]
    gs = [synth.normal_codes(n, 8601, i, std_codes=40) for i, n in enumerate(sizes)]
    pgs = [-19, -13, -16]
    m_d = [G.dev(m) for m in masters]
    w_d = [G.zeros(n, torch.int8) for n in sizes]
    step = G.dev(np.array([2], dtype=np.int64))
    cur = [m.copy() for m in masters]
    for it in range(3):
        eoq.eoq_update_wide(G.handle(), m_d, w_d, [G.dev(g) for g in gs], [G.dev(np.array([p], dtype=np.int32)) for p in pgs], 37, -5,
                            k_u, k_m, eoq.EOQ_ROUND_STOCHASTIC if stochastic else eoq.EOQ_ROUND_RNE, seed=13, step_dev=step)
        assert G.status_clear() == 0
        for i in range(len(sizes)):
            cur[i], w8, _, _ = oracle.update_k(cur[i], gs[i], pgs[i], 37, -5, k_u, k_m, stochastic=stochastic, seed=13, step=2 + it, tensor_id=i)
            assert np.array_equal(G.host(m_d[i]), cur[i]), (it, i, "master")
            assert np.array_equal(G.host(w_d[i]), w8), (it, i, "w")
    assert step.item() == 5

"""The weight gradient in two parts (eoq_conv_wgrad_gemm per layer, one eoq_wgrad_finish for all layers) against the
oracle and against the one-call form, bit for bit: both GEMM kernels, with and without the b1 term, more layers than
one launch batch holds."""
import numpy as np
import pytest
import torch

import oracle
from oracle import ConvDesc
from paper_2105_13890_b200 import eoq, synth

import gpu_util as G

pytestmark = pytest.mark.gpu

LAYERS = [  # n, h, w, c_in, c_out, k, stride, pad, b1 (None: no bias in front of the convolution)
    (2, 12, 12, 32, 32, 3, 1, 1, -2),       # patch kernel, int32 slices
    (3, 7, 7, 64, 128, 3, 1, 1, 5),
    (2, 10, 10, 32, 64, 3, 2, 1, 3),        # strided: per-tap kernel, int64 sums
    (2, 9, 11, 48, 32, 1, 1, 0, -7),
    (2, 16, 16, 16, 32, 7, 2, 3, None),     # a first-layer shape
    (1, 20, 20, 64, 64, 5, 1, 2, 0),        # b1 present and zero
]


def make(case, seed):
    n, h, w, c_in, c_out, k, stride, pad, b1 = case
    d = ConvDesc(n, h, w, c_in, c_out, k, k, stride, pad)
    e3 = synth.normal_codes((n, d.ho, d.wo, c_out), seed, 0)
    x0 = synth.relu_codes((n, h, w, c_in), seed, 1)
    S = oracle.conv_wgrad_acc(d, e3, x0, b1 or 0)
    g_o, pg_o, _ = oracle.sq_int(S, -12 - 7)
    return d, e3, x0, b1, g_o, pg_o


@pytest.mark.parametrize("repeat", [1, 4])     # 6 and 24 layers: the second needs two launch batches
def test_gemm_per_layer_and_one_finish_for_all(repeat):
    hd = G.handle()
    cases = [make(c, 8900 + 10 * r + i) for r in range(repeat) for i, c in enumerate(LAYERS)]
    descs, e3s, pes, b1s, gs, pgs, wss, parts = [], [], [], [], [], [], [], []
    for d, e3, x0, b1, _, _ in cases:
        gd = G.gdesc(d)
        ws = G.workspace(gd, eoq.EOQ_PASS_WGRAD)
        e3_d, pe = G.dev(e3), G.dev(np.array([-12], dtype=np.int32))
        parts.append(eoq.eoq_conv_wgrad_gemm(hd, gd, e3_d, pe, G.dev(x0), ws))
        descs.append(gd); e3s.append(e3_d); pes.append(pe); wss.append(ws)
        b1s.append(None if b1 is None else G.dev(np.array([b1], dtype=np.int32)))
        gs.append(G.zeros((d.c_out, d.kh, d.kw, d.c_in), torch.int8)); pgs.append(G.zeros(1, torch.int32))
    eoq.eoq_wgrad_finish(hd, descs, e3s, pes, b1s, gs, pgs, wss, parts)
    torch.cuda.synchronize()
    assert eoq.eoq_last_status(hd) == 0
    for (d, e3, x0, b1, g_o, pg_o), g, pg in zip(cases, gs, pgs):
        assert np.array_equal(G.host(g), g_o) and pg.item() == pg_o, (d, b1)
    # the same through the one-call form, on the same handle (its cells are clean)
    d, e3, x0, b1, g_o, pg_o = cases[0]
    gd = G.gdesc(d)
    g1, pg1 = G.zeros(g_o.shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_conv_wgrad_dev(hd, gd, G.dev(e3), G.dev(np.array([-12], dtype=np.int32)), G.dev(x0), G.dev(np.array([b1], dtype=np.int32)), g1, pg1,
                           G.workspace(gd, eoq.EOQ_PASS_WGRAD))
    torch.cuda.synchronize()
    assert np.array_equal(G.host(g1), g_o) and pg1.item() == pg_o


def test_a_zero_error_gives_zero_gradients_and_the_flag():
    hd = G.handle()
    d = ConvDesc(2, 8, 8, 32, 32, 3, 3, 1, 1)
    gd = G.gdesc(d)
    ws = G.workspace(gd, eoq.EOQ_PASS_WGRAD)
    e3, pe = G.zeros((2, 8, 8, 32), torch.int8), G.dev(np.array([-12], dtype=np.int32))
    parts = eoq.eoq_conv_wgrad_gemm(hd, gd, e3, pe, G.dev(synth.relu_codes((2, 8, 8, 32), 1, 0)), ws)
    g, pg = G.empty((32, 3, 3, 32), torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_wgrad_finish(hd, [gd], [e3], [pe], [G.dev(np.array([4], dtype=np.int32))], [g], [pg], [ws], [parts])
    torch.cuda.synchronize()
    assert not G.host(g).any() and pg.item() == -19
    assert eoq.eoq_last_status(hd) == eoq.EOQ_DEV_SQ_ZERO
    G.status_clear()

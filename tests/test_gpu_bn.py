"""Batch normalisation behind the convolution on the GPU (eoq_bn_fwd / eoq_bn_bwd, the comparison case of Sec. 5.3)
against the oracle, bit for bit: codes, mask bits, the per-channel constants, the fp32 error and parameter gradients,
and the int8 error after Q_e."""
import numpy as np
import pytest
import torch

import oracle
from oracle import ConvDesc
from paper_2105_13890_b200 import eoq, synth

import gpu_util as G

pytestmark = pytest.mark.gpu

RECORD = np.dtype([("s1", "i8"), ("shh", "i8"), ("shl", "i8"), ("sll", "i8"), ("d1", "i8"), ("d2", "i8"), ("mu", "f8"), ("inv", "f8"),
                   ("scale", "f4"), ("shift", "f4"), ("ca", "f4"), ("cb", "f4"), ("cc", "f4"), ("pad", "f4")])


def run_bn(acc, p, gamma, beta, eps, E, p_e):
    """Forward and backward on the GPU for int32 sums acc [n,h,w,c]."""
    hd = G.handle()
    c = acc.shape[-1]
    P = acc.size // c
    ws = G.zeros(eoq.eoq_bn_workspace_size(c), torch.uint8)
    acc_d = G.dev(acc.astype(np.int32))
    g_d, b_d = G.dev(gamma), G.dev(beta)
    x5, mask = G.zeros(acc.shape, torch.int8), G.zeros((acc.size + 7) // 8, torch.uint8)
    eoq.eoq_bn_fwd(hd, acc_d, p, P, c, g_d, b_d, eps, x5, mask, ws)
    torch.cuda.synchronize()
    rec_fwd = G.host(ws)[: RECORD.itemsize * c].view(RECORD).copy()
    da = G.zeros(acc.shape, torch.float32)
    dgamma, dbeta = G.zeros(c, torch.float32), G.zeros(c, torch.float32)
    eoq.eoq_bn_bwd(hd, G.dev(E), G.dev(np.array([p_e], dtype=np.int32)), mask, acc_d, p, P, c, g_d, ws, da, dgamma, dbeta)
    e8, pe8 = G.zeros(acc.shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_quantize(hd, eoq.EOQ_SQ, da, True, None, acc.size, e8, pe8)
    torch.cuda.synchronize()
    assert eoq.eoq_last_status(hd) == 0
    return {"x5": G.host(x5), "mask": G.unpack_mask(mask, acc.shape), "rec": rec_fwd, "da": G.host(da), "dgamma": G.host(dgamma),
            "dbeta": G.host(dbeta), "e8": G.host(e8), "pe8": pe8.item()}


def check(acc, p, gamma, beta, eps, E, p_e):
    got = run_bn(acc, p, gamma, beta, eps, E, p_e)
    r = oracle.bn_forward(acc, p, gamma, beta, eps)
    assert np.array_equal(got["rec"]["mu"], r["ch"]["mu"]) and np.array_equal(got["rec"]["inv"], r["ch"]["inv"])
    assert np.array_equal(got["rec"]["scale"], r["ch"]["scale"]) and np.array_equal(got["rec"]["shift"], r["ch"]["shift"])
    assert np.array_equal(got["x5"], r["x5"]) and np.array_equal(got["mask"], r["mask"])
    da, dgamma, dbeta = oracle.bn_backward(E, p_e, r["mask"], acc, p, gamma, r["ch"])
    assert np.array_equal(got["dgamma"], dgamma) and np.array_equal(got["dbeta"], dbeta)
    assert np.array_equal(got["da"], da)
    codes, p_out, _ = oracle.quantize_f32(oracle.MODE_SQ, da)
    assert np.array_equal(got["e8"], codes) and got["pe8"] == p_out


@pytest.mark.parametrize("n,h,w,c_in,c_out,k", [(4, 12, 12, 32, 32, 3), (3, 9, 7, 64, 48, 3), (2, 8, 8, 16, 16, 1), (5, 14, 14, 64, 256, 3)])
def test_batch_norm_behind_a_convolution(n, h, w, c_in, c_out, k):
    d = ConvDesc(n, h, w, c_in, c_out, k, k, 1, k // 2)
    x0 = synth.relu_codes((n, h, w, c_in), 8700 + c_out, 0)
    wt = synth.int8_uniform((c_out, k, k, c_in), 8700 + c_out, 1, -40, 40)
    hd = G.handle()
    gd = G.gdesc(d)
    shape = (n, d.ho, d.wo, c_out)
    x5, mask = G.zeros(shape, torch.int8), G.zeros((int(np.prod(shape)) + 7) // 8, torch.uint8)
    acc = G.zeros(shape, torch.int32)
    eoq.eoq_conv_fwd(hd, gd, G.dev(x0), None, 0, G.dev(wt), 128, 0, None, True, x5, None, mask, acc, G.workspace(gd, eoq.EOQ_PASS_FWD))
    torch.cuda.synchronize()
    A = oracle.conv_fwd_acc(d, x0, 0, wt)
    assert np.array_equal(G.host(acc).astype(np.int64), A)
    rng = np.random.default_rng(c_out)
    gamma = rng.uniform(0.5, 1.5, c_out).astype(np.float32)
    beta = rng.normal(0, 0.3, c_out).astype(np.float32)
    E = synth.normal_codes(shape, 8700 + c_out, 2)
    check(A, -14, gamma, beta, 1e-5, E, -12)


def test_large_sums_and_a_constant_channel():
    """Sums near the int32 limits (the three-part squares carry), a channel without variance, a channel of zeros."""
    rng = np.random.default_rng(77)
    shape = (3, 10, 11, 32)
    A = rng.integers(-2 ** 30, 2 ** 30, shape).astype(np.int64)
    A[..., 1] = 2 ** 30 + rng.integers(-3, 4, shape[:-1])     # large mean, tiny spread: the variance cancels 58 bits
    A[..., 2] = -123456
    A[..., 3] = 0
    A[..., 4] = rng.choice([-2 ** 31, 2 ** 31 - 1], shape[:-1])
    c = shape[-1]
    gamma = np.linspace(0.25, 2.0, c).astype(np.float32)
    beta = np.linspace(-1, 1, c).astype(np.float32)
    E = synth.normal_codes(shape, 8800, 0)
    check(A, -30, gamma, beta, 1e-5, E, -9)


def test_argument_errors():
    hd = G.handle()
    ws = G.zeros(eoq.eoq_bn_workspace_size(16), torch.uint8)
    acc = G.zeros((4, 16), torch.int32)
    g = G.zeros(16, torch.float32)
    x5, mask = G.zeros((4, 16), torch.int8), G.zeros(8, torch.uint8)
    with pytest.raises(eoq.EoqError):
        eoq.eoq_bn_fwd(hd, acc, -14, 4, 24, g, g, 1e-5, x5, mask, ws)         # channels not a multiple of 16
    with pytest.raises(eoq.EoqError):
        eoq.eoq_bn_fwd(hd, acc, -14, 0, 16, g, g, 1e-5, x5, mask, ws)         # no pixels
    with pytest.raises(eoq.EoqError):
        eoq.eoq_bn_fwd(hd, acc, -14, 4, 16, g, g, 1e-5, x5, mask, ws[:64])    # workspace too small

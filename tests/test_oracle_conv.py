"""Pins for the oracle's three convolutions: brute force, a float64 library convolution, adjoint identities."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import ConvDesc
from paper_2105_13890_b200 import synth

SHAPES = [
    ConvDesc(2, 5, 6, 3, 4, 3, 3, 1, 1),
    ConvDesc(1, 7, 7, 2, 3, 3, 3, 2, 1),
    ConvDesc(2, 6, 5, 4, 2, 1, 1, 1, 0),
    ConvDesc(2, 6, 6, 4, 2, 1, 1, 2, 0),
    ConvDesc(1, 9, 8, 2, 2, 7, 7, 2, 3),
    ConvDesc(1, 4, 4, 1, 1, 3, 3, 1, 0),
    ConvDesc(1, 2, 2, 2, 2, 3, 3, 1, 1),
]


def data(d, seed):
    x0 = synth.int8_uniform((d.n, d.h, d.w, d.c_in), seed, 0)
    w = synth.int8_uniform((d.c_out, d.kh, d.kw, d.c_in), seed, 1)
    e3 = synth.int8_uniform((d.n, d.ho, d.wo, d.c_out), seed, 2)
    return x0, w, e3


def brute_fwd(d, x0, b1, w):
    A = np.zeros((d.n, d.ho, d.wo, d.c_out), dtype=object)
    for n in range(d.n):
        for y in range(d.ho):
            for x in range(d.wo):
                for oc in range(d.c_out):
                    s = 0
                    for kh in range(d.kh):
                        for kw in range(d.kw):
                            iy, ix = y * d.stride + kh - d.pad, x * d.stride + kw - d.pad
                            if 0 <= iy < d.h and 0 <= ix < d.w:
                                for ic in range(d.c_in):
                                    s += (int(x0[n, iy, ix, ic]) + b1) * int(w[oc, kh, kw, ic])
                    A[n, y, x, oc] = s
    return A.astype(np.int64)


@pytest.mark.parametrize("d", SHAPES[:5])
@pytest.mark.parametrize("b1", [0, -3])
def test_fwd_matches_brute_force(d, b1):
    x0, w, _ = data(d, 11)
    assert np.array_equal(oracle.conv_fwd_acc(d, x0, b1, w), brute_fwd(d, x0, b1, w))


def to_nchw(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch.float64).permute(0, 3, 1, 2).contiguous()


def x1_dense(d, x0, b1):
    # x1 laid out with an explicit zero halo, so the library call below uses padding=0
    x1 = np.zeros((d.n, d.h + 2 * d.pad, d.w + 2 * d.pad, d.c_in), dtype=np.int64)
    x1[:, d.pad:d.pad + d.h, d.pad:d.pad + d.w, :] = x0.astype(np.int64) + b1
    return x1


@pytest.mark.parametrize("d", SHAPES + [ConvDesc(2, 12, 12, 16, 16, 3, 3, 1, 1), ConvDesc(2, 12, 12, 16, 32, 3, 3, 2, 1)])
@pytest.mark.parametrize("b1", [0, 5])
def test_all_three_match_float64_library_convolution(d, b1):
    """Sums stay far below 2^53, so a float64 convolution is exact and pins index order, signs and transposes."""
    x0, w, e3 = data(d, 12)
    xt = to_nchw(x1_dense(d, x0, b1)).requires_grad_(True)
    wt = to_nchw(w).requires_grad_(True)  # [oc, ic, kh, kw]
    y = F.conv2d(xt, wt, stride=d.stride, padding=0)
    A = oracle.conv_fwd_acc(d, x0, b1, w)
    assert np.array_equal(y.detach().permute(0, 2, 3, 1).numpy().astype(np.int64), A)
    y.backward(to_nchw(e3))
    gx = xt.grad.permute(0, 2, 3, 1).numpy().astype(np.int64)[:, d.pad:d.pad + d.h, d.pad:d.pad + d.w, :]
    gw = wt.grad.permute(0, 2, 3, 1).numpy().astype(np.int64)
    assert np.array_equal(oracle.conv_dgrad_acc(d, e3, w), gx)
    assert np.array_equal(oracle.conv_wgrad_acc(d, e3, x0, b1), gw)


@pytest.mark.parametrize("d", SHAPES)
def test_adjoint_identities_hold_exactly(d):
    """<conv(x1, w), e> = <x1, dgrad(e, w)> = <w, wgrad(e, x1)> on the pre-quantization integers."""
    x0, w, e3 = data(d, 13)
    b1 = 2
    A = oracle.conv_fwd_acc(d, x0, b1, w)
    B = oracle.conv_dgrad_acc(d, e3, w)
    G = oracle.conv_wgrad_acc(d, e3, x0, b1)
    lhs = int((A * e3.astype(np.int64)).sum())
    assert lhs == int(((x0.astype(np.int64) + b1) * B).sum())
    assert lhs == int((w.astype(np.int64) * G).sum())


def test_identity_kernel_reproduces_input():
    d = ConvDesc(1, 5, 5, 3, 3, 3, 3, 1, 1)
    x0 = synth.int8_uniform((1, 5, 5, 3), 14, 0)
    w = np.zeros((3, 3, 3, 3), dtype=np.int8)
    for c in range(3):
        w[c, 1, 1, c] = 64
    A = oracle.conv_fwd_acc(d, x0, 7, w)
    assert np.array_equal(A, (x0.astype(np.int64) + 7) * 64)

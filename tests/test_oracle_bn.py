"""Pins of the oracle's batch normalisation (the comparison case of Sec. 5.3) to a library routine and to what the
definition fixes: the float64 library batch-norm and its autograd backward, invariants of the statistics, the exponent
bookkeeping, and the exactness of the integer sums."""
import numpy as np
import pytest
import torch

import oracle


def conv_like(shape, seed, spread=4000):
    rng = np.random.default_rng(seed)
    c = shape[-1]
    # channels with different means and spreads, as a convolution output has
    return (rng.normal(0, 1, shape) * rng.uniform(0.2, 1.0, c) * spread + rng.normal(0, spread / 3, c)).round().astype(np.int64)


def library_bn(A, p, gamma, beta, eps):
    a = torch.tensor(A.astype(np.float64) * 2.0 ** p, dtype=torch.float64, requires_grad=True)
    g = torch.tensor(gamma, dtype=torch.float64, requires_grad=True)
    b = torch.tensor(beta, dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.batch_norm(a.permute(0, 3, 1, 2), None, None, g, b, training=True, eps=eps).permute(0, 2, 3, 1)
    return a, g, b, y


@pytest.mark.parametrize("shape,p", [((4, 6, 5, 16), -14), ((2, 3, 3, 32), -9), ((8, 1, 1, 16), -14)])
def test_forward_matches_the_library_batch_norm(shape, p):
    A = conv_like(shape, 31)
    c = shape[-1]
    gamma = np.linspace(0.5, 1.5, c).astype(np.float32)
    beta = np.linspace(-0.2, 0.3, c).astype(np.float32)
    r = oracle.bn_forward(A, p, gamma, beta, 1e-5)
    _, _, _, y = library_bn(A, p, gamma, beta, 1e-5)
    y = y.detach().numpy()
    assert np.allclose(r["y"], y, rtol=2e-6, atol=2e-6)
    assert np.array_equal(r["mask"], (r["y"] > 0).astype(np.uint8))
    # Q_a2 of relu(y): the library's value decides the code wherever it is not within rounding noise of a tie
    t = np.clip(y, 0, None) * 128
    want = np.minimum(np.rint(t), 127)
    clear = np.abs(t - np.floor(t) - 0.5) > 1e-3
    assert np.array_equal(r["x5"][clear], want[clear].astype(np.int8))
    assert clear.mean() > 0.95


def test_backward_matches_the_library_autograd():
    shape, p, p_e = (4, 5, 6, 16), -14, -11
    A = conv_like(shape, 32)
    c = shape[-1]
    gamma = np.linspace(0.7, 1.3, c).astype(np.float32)
    beta = np.linspace(-0.1, 0.2, c).astype(np.float32)
    E = np.random.default_rng(5).integers(-127, 128, shape).astype(np.int8)
    r = oracle.bn_forward(A, p, gamma, beta, 1e-5)
    da, dgamma, dbeta = oracle.bn_backward(E, p_e, r["mask"], A, p, gamma, r["ch"])
    a, g, b, y = library_bn(A, p, gamma, beta, 1e-5)
    dy = torch.tensor(E.astype(np.float64) * 2.0 ** p_e * r["mask"])     # straight through the clamp, gated by the ReLU
    y.backward(dy)
    scale = np.abs(a.grad.numpy()).max()
    assert np.allclose(da, a.grad.numpy(), rtol=1e-4, atol=1e-5 * scale)
    assert np.allclose(dgamma, g.grad.numpy(), rtol=1e-5, atol=1e-6)
    assert np.allclose(dbeta, b.grad.numpy(), rtol=1e-6, atol=1e-7)
    # a planted mistake is seen: without the ReLU gate the result differs
    da2, _, dbeta2 = oracle.bn_backward(E, p_e, np.ones_like(r["mask"]), A, p, gamma, r["ch"])
    assert not np.allclose(dbeta2, b.grad.numpy(), rtol=1e-3, atol=1e-4)


def test_statistics_invariants_and_special_cases():
    shape, p = (3, 4, 4, 16), -12
    A = conv_like(shape, 33)
    c = shape[-1]
    one, zero = np.ones(c, dtype=np.float32), np.zeros(c, dtype=np.float32)
    y = oracle.bn_forward(A, p, one, zero, 0.0)["y"].astype(np.float64)
    assert np.allclose(y.mean(axis=(0, 1, 2)), 0, atol=1e-6) and np.allclose(y.var(axis=(0, 1, 2)), 1, rtol=1e-5)
    # a constant channel has zero variance: y = beta there (eps keeps the division finite), up to the single-precision
    # rounding of scale * a + shift, whose two terms cancel
    B = A.copy()
    B[..., 3] = 1234
    beta = np.full(c, 0.25, dtype=np.float32)
    r = oracle.bn_forward(B, p, one, beta, 1e-5)
    assert np.allclose(r["y"][..., 3], 0.25, atol=2e-5) and np.all(r["x5"][..., 3] == 32)
    # the same values written at another exponent give the same bits (2A at p - 1 is A at p)
    r1 = oracle.bn_forward(A, p, one, beta, 1e-5)
    r2 = oracle.bn_forward(2 * A, p - 1, one, beta, 1e-5)
    assert np.array_equal(r1["y"], r2["y"]) and np.array_equal(r1["x5"], r2["x5"])
    # shifting a channel by a constant changes nothing but its mean
    S = A.copy()
    S[..., 5] += 4096
    r3 = oracle.bn_forward(S, p, one, beta, 1e-5)
    assert np.allclose(r3["y"][..., 5], r1["y"][..., 5], atol=2e-6) and r3["ch"]["mu"][5] == r1["ch"]["mu"][5] + 4096


def test_sums_are_exact_where_double_precision_would_not_be():
    """Large codes with a small spread: sum(A^2)/P - mean^2 cancels 40 bits; the 128-bit sums keep the variance exact."""
    rng = np.random.default_rng(34)
    shape, p = (4, 8, 8, 16), -30
    A = (2 ** 30 + rng.integers(-3, 4, shape)).astype(np.int64)
    r = oracle.bn_forward(A, p, np.ones(16, dtype=np.float32), np.zeros(16, dtype=np.float32), 0.0)
    d = (A - A.mean(axis=(0, 1, 2))).astype(np.float64)
    want = d / np.sqrt((d * d).mean(axis=(0, 1, 2)))
    # the per-element step runs in single precision on (float)A, which cannot hold 2^30 + 3: only the statistics are checked
    var_exact = (d * d).mean(axis=(0, 1, 2)) * 4.0 ** p
    assert np.allclose(1.0 / r["ch"]["inv"] ** 2, var_exact, rtol=1e-12)
    assert np.isfinite(want).all()

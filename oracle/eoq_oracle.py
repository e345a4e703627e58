"""ctypes front end of the EOQ oracle (test infrastructure, not product code).

The arithmetic lives in ``eoq_oracle.c`` (plain direct loops, int64); this file
compiles it with gcc, marshals numpy arrays, and composes the per-layer forward
and backward chains of Sec. 3.2.1 of arXiv 2105.13890 out of those pieces in the
paper's order.  Nothing here is shared with, or calls, the CUDA path.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "eoq_oracle.c")
_SO = os.path.join(_HERE, "_eoq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle next to its source (gcc, OpenMP, no FMA contraction)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _SO)
    return _SO


class _ConvT(C.Structure):
    _fields_ = [(k, C.c_int) for k in ("n", "h", "w", "c_in", "c_out", "kh", "kw", "stride", "pad")]


@dataclass(frozen=True)
class ConvDesc:
    """Geometry of one convolution layer (square stride and padding)."""

    n: int
    h: int
    w: int
    c_in: int
    c_out: int
    kh: int
    kw: int
    stride: int = 1
    pad: int = 0

    @property
    def ho(self) -> int:
        return (self.h + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def wo(self) -> int:
        return (self.w + 2 * self.pad - self.kw) // self.stride + 1

    def _c(self) -> _ConvT:
        return _ConvT(self.n, self.h, self.w, self.c_in, self.c_out, self.kh, self.kw, self.stride, self.pad)


def _L():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.eoq_o_rne_shr.restype = C.c_int64
        lib.eoq_o_rne_shr.argtypes = [C.c_int64, C.c_int]
        lib.eoq_o_q_code.restype = C.c_int64
        lib.eoq_o_q_code.argtypes = [C.c_double]
        lib.eoq_o_cq_code.restype = C.c_int64
        lib.eoq_o_cq_code.argtypes = [C.c_double]
        lib.eoq_o_round_log2_u64.restype = C.c_int
        lib.eoq_o_round_log2_u64.argtypes = [C.c_uint64]
        lib.eoq_o_update_hash.restype = C.c_uint64
        lib.eoq_o_update_hash.argtypes = [C.c_uint64] * 4
        lib.eoq_o_expf.restype = C.c_float
        lib.eoq_o_expf.argtypes = [C.c_float]
        lib.eoq_o_join.restype = C.c_int
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _i8(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int8)


# --------------------------------------------------------------------------- quantizers (Sec. 3.2.2)

def rne_shr(a: int, s: int) -> int:
    """R(a / 2^s), nearest with ties to even; s < 0 multiplies by 2^-s."""
    return int(_L().eoq_o_rne_shr(int(a), int(s)))


def q_code(x: float) -> int:
    """Code of Q(x, 8): R(x * 2^7)."""
    return int(_L().eoq_o_q_code(float(x)))


def cq_code(x: float) -> int:
    """Code of CQ(x, 8): the Q code clamped to [-127, 127]."""
    return int(_L().eoq_o_cq_code(float(x)))


def round_log2(m: int) -> int:
    """R(log2 m) for a positive integer m (the exponent of scale(x))."""
    return int(_L().eoq_o_round_log2_u64(int(m)))


def sq_int(a, p_a: int):
    """SQ(., 8) of integer codes a at exponent p_a -> (int32 codes, p_out, zero flag)."""
    a = np.ascontiguousarray(a, dtype=np.int64)
    codes = np.empty(a.shape, dtype=np.int32)
    p_out = C.c_int(0)
    z = _L().eoq_o_sq_i64(_p(a), C.c_size_t(a.size), C.c_int(p_a), _p(codes), C.byref(p_out))
    return codes, p_out.value, int(z)


MODE_Q, MODE_CQ, MODE_SQ = 0, 1, 2


def quantize_f32(mode: int, x):
    """Q / CQ / SQ of an fp32 tensor -> (int32 codes, exponent, flag); flag -1 = non-finite input."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    codes = np.empty(x.shape, dtype=np.int32)
    p_out = C.c_int(0)
    z = _L().eoq_o_quantize_f32(C.c_int(mode), _p(x), C.c_size_t(x.size), _p(codes), C.byref(p_out))
    return codes, p_out.value, int(z)


# --------------------------------------------------------------------------- convolutions (Sec. 3.2.1)

def conv_fwd_acc(d: ConvDesc, x0, b1_c: int, w) -> np.ndarray:
    """conv(x0 + b1) with zero halo: int64 accumulators [n, ho, wo, c_out]."""
    x0, w = _i8(x0), _i8(w)
    assert x0.shape == (d.n, d.h, d.w, d.c_in) and w.shape == (d.c_out, d.kh, d.kw, d.c_in)
    A = np.empty((d.n, d.ho, d.wo, d.c_out), dtype=np.int64)
    dc = d._c()
    _L().eoq_o_conv_fwd_acc(C.byref(dc), _p(x0), C.c_int(b1_c), _p(w), _p(A))
    return A


def conv_dgrad_acc(d: ConvDesc, e3, w) -> np.ndarray:
    """Transposed convolution of the error: int64 accumulators [n, h, w, c_in]."""
    e3, w = _i8(e3), _i8(w)
    assert e3.shape == (d.n, d.ho, d.wo, d.c_out) and w.shape == (d.c_out, d.kh, d.kw, d.c_in)
    B = np.empty((d.n, d.h, d.w, d.c_in), dtype=np.int64)
    dc = d._c()
    _L().eoq_o_conv_dgrad_acc(C.byref(dc), _p(e3), _p(w), _p(B))
    return B


def conv_wgrad_acc(d: ConvDesc, e3, x0, b1_c: int) -> np.ndarray:
    """Correlation of the error with x1 = x0 + b1: int64 accumulators [c_out, kh, kw, c_in]."""
    e3, x0 = _i8(e3), _i8(x0)
    assert e3.shape == (d.n, d.ho, d.wo, d.c_out) and x0.shape == (d.n, d.h, d.w, d.c_in)
    G = np.empty((d.c_out, d.kh, d.kw, d.c_in), dtype=np.int64)
    dc = d._c()
    _L().eoq_o_conv_wgrad_acc(C.byref(dc), _p(e3), _p(x0), C.c_int(b1_c), _p(G))
    return G


def fwd_epilogue(A, acc_shift: int, gamma_c: int, b2_c: int, shortcut=None, relu: bool = True):
    """x2, x5 and the ReLU mask from the conv accumulator (forward chain, steps x2..x5)."""
    A = np.ascontiguousarray(A, dtype=np.int64)
    x2 = np.empty(A.shape, dtype=np.int32)
    x5 = np.empty(A.shape, dtype=np.int8)
    mask = np.empty(A.shape, dtype=np.uint8)
    sc = None if shortcut is None else _i8(shortcut)
    if sc is not None:
        assert sc.shape == A.shape
    _L().eoq_o_fwd_epilogue(_p(A), C.c_size_t(A.size), C.c_int(acc_shift), C.c_int(gamma_c), C.c_int(b2_c),
                            _p(sc) if sc is not None else None, C.c_int(1 if relu else 0), _p(x2), _p(x5), _p(mask))
    return x2, x5, mask


def layer_forward(d: ConvDesc, x0, b1_c: int, w, gamma_c: int, b2_c: int, shortcut=None, relu: bool = True,
                  x_exp: int = -7):
    """Forward chain x0 -> x5 of one layer (Sec. 3.2.1).

    x_exp is the exponent of x0 (-7 everywhere but at the network input, whose SQ
    exponent moves the Q_a1 shift to -x_exp bits).
    """
    A = conv_fwd_acc(d, x0, b1_c, w)
    x2, x5, mask = fwd_epilogue(A, -x_exp, gamma_c, b2_c, shortcut, relu)
    return {"acc": A, "x2": x2, "x5": x5, "mask": mask}


def err_prescale(e0, p0: int, mask, x2, gamma_c: int):
    """e1 = e0 * mask, e3 = Q_e(gamma * e1), plus sum(e1) and sum(e1 * x2)."""
    e0 = _i8(e0)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    x2c = None if x2 is None else np.ascontiguousarray(x2, dtype=np.int32)
    e3 = np.empty(e0.shape, dtype=np.int32)
    p3 = C.c_int(0)
    s1 = C.c_int64(0)
    s2 = C.c_int64(0)
    z = _L().eoq_o_err_prescale(_p(e0), C.c_int(p0), _p(mask), _p(x2c) if x2c is not None else None,
                                C.c_size_t(e0.size), C.c_int(gamma_c), _p(e3), C.byref(p3), C.byref(s1), C.byref(s2))
    return e3.astype(np.int8), p3.value, int(s1.value), int(s2.value), int(z)


def layer_backward(d: ConvDesc, e0, p0: int, mask, x2, x0, b1_c: int, w, gamma_c: int):
    """Error chain e0 -> e4 and the four gradients of one layer (Sec. 3.2.1)."""
    e3, p3, s_e1, s_e1x2, _ = err_prescale(e0, p0, mask, x2, gamma_c)
    B = conv_dgrad_acc(d, e3, w)
    e4, p4, z4 = sq_int(B, p3 - 7)
    G = conv_wgrad_acc(d, e3, x0, b1_c)
    g_w, p_gw, zg = sq_int(G, p3 - 7)
    g_b1, p_b1, _ = sq_int(np.array([int(e4.astype(np.int64).sum())]), p4)
    g_b2, p_b2, _ = sq_int(np.array([s_e1]), p0)
    g_ga, p_ga, _ = sq_int(np.array([s_e1x2]), p0 - 7)
    return {
        "e3": e3, "p3": p3, "dgrad_acc": B, "e4": e4.astype(np.int8), "p4": p4, "e4_zero": z4,
        "wgrad_acc": G, "g_w": g_w.astype(np.int8), "p_gw": p_gw, "g_w_zero": zg,
        "sum_e4": int(e4.astype(np.int64).sum()), "sum_e1": s_e1, "sum_e1x2": s_e1x2,
        "g_b1": (int(g_b1[0]), p_b1), "g_b2": (int(g_b2[0]), p_b2), "g_gamma": (int(g_ga[0]), p_ga),
    }


# --------------------------------------------------------------------------- update (Sec. 3.2.3)

def update_hash(seed: int, step: int, tensor_id: int, idx: int) -> int:
    return int(_L().eoq_o_update_hash(seed, step, tensor_id, idx))


def update(theta, g, p_g: int, lr_mant: int, lr_exp: int, lo: int = -127, hi: int = 127, stochastic: bool = False,
           seed: int = 0, step: int = 0, tensor_id: int = 0):
    """theta <- sat(theta - align(SQ(lr * g)), lo, hi) -> (new int32 codes, exponent of u, zero flag)."""
    th = np.array(theta, dtype=np.int32).reshape(-1).copy()
    g = _i8(g).reshape(-1)
    assert th.size == g.size
    p_u = C.c_int(0)
    z = _L().eoq_o_update(_p(th), _p(g), C.c_int(p_g), C.c_size_t(th.size), C.c_int(lr_mant), C.c_int(lr_exp),
                          C.c_int(lo), C.c_int(hi), C.c_int(1 if stochastic else 0), C.c_uint64(seed),
                          C.c_uint64(step), C.c_uint64(tensor_id), C.byref(p_u))
    return th.reshape(np.shape(theta)), p_u.value, int(z)


# --------------------------------------------------------------------------- Fixup initialisation (Sec. 3.1)

def fixup_alpha(L: int, m: int) -> float:
    """Layer-wise coefficient L^(-1/(2m-2)) of Eq. (1); L residual blocks, m layers per block."""
    return float(L) ** (-1.0 / (2 * m - 2))


def kaiming_std(fan_in: int) -> float:
    """Standard deviation of the Kaiming normal N(0, 2/n), n inputs per output (Sec. 4)."""
    return float(np.sqrt(2.0 / fan_in))


def fixup_weights_f32(z, fan_in: int, L: int, m: int, in_branch: bool = True) -> np.ndarray:
    """fp32 weights from standard normal draws z: Kaiming std, times alpha inside residual branches."""
    s = kaiming_std(fan_in) * (fixup_alpha(L, m) if in_branch else 1.0)
    return (np.asarray(z, dtype=np.float64) * s).astype(np.float32)


def q_w(w_f32) -> np.ndarray:
    """Q_w = CQ(., 8): int8 weight codes."""
    codes, _, flag = quantize_f32(MODE_CQ, w_f32)
    assert flag == 0
    return codes.astype(np.int8)


# --------------------------------------------------------------------------- network glue (conventions of this build)

def maxpool_fwd(x, k: int, s: int, p: int):
    """Max-pooling on int8 codes -> (codes [n,ho,wo,c], flat NHWC index of the first maximum per output)."""
    x = _i8(x)
    n, h, w, c = x.shape
    ho, wo = (h + 2 * p - k) // s + 1, (w + 2 * p - k) // s + 1
    y = np.empty((n, ho, wo, c), dtype=np.int8)
    idx = np.empty((n, ho, wo, c), dtype=np.int64)
    _L().eoq_o_maxpool_fwd(_p(x), C.c_int(n), C.c_int(h), C.c_int(w), C.c_int(c), C.c_int(k), C.c_int(s), C.c_int(p), _p(y), _p(idx))
    return y, idx


def maxpool_bwd(e, idx, in_shape) -> np.ndarray:
    """Exact sums of the error codes routed to the argmax positions: int64 [in_shape]."""
    e = _i8(e)
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    S = np.zeros(in_shape, dtype=np.int64)
    _L().eoq_o_maxpool_bwd(_p(e), _p(idx), C.c_size_t(e.size), _p(S))
    return S


def avgpool_sum(x) -> np.ndarray:
    """Integer sum over the spatial positions per (sample, channel): int64 [n, c]."""
    x = _i8(x)
    n, h, w, c = x.shape
    sums = np.empty((n, c), dtype=np.int64)
    _L().eoq_o_avgpool_sum(_p(x), C.c_int(n), C.c_int(h * w), C.c_int(c), _p(sums))
    return sums


def join(a, pa: int, b, pb: int, mask_b=None):
    """Exact sum of two error tensors at the smaller exponent -> (int64 sums, exponent); mask_b gates b."""
    a, b = _i8(a), _i8(b)
    assert a.shape == b.shape
    S = np.empty(a.shape, dtype=np.int64)
    m = None if mask_b is None else np.ascontiguousarray(mask_b, dtype=np.uint8)
    p = _L().eoq_o_join(_p(a), C.c_int(pa), _p(b), C.c_int(pb), _p(m) if m is not None else None, C.c_size_t(a.size), _p(S))
    return S, int(p)


def expf(x: float) -> float:
    """The head's own exp in fp32 (fused multiply-adds and a power-of-two scaling only)."""
    return float(_L().eoq_o_expf(C.c_float(x)))


def head(sums, hw: int, W, bias, labels, lr: float):
    """The floating-point last layer: pooling scale, linear layer, softmax cross-entropy (mean), its gradient
    with respect to the pooled activations, and the SGD step of W and bias (in place).
    -> (loss, dpooled fp32 [n, c], logits fp32 [n, classes])."""
    sums = np.ascontiguousarray(sums, dtype=np.int64)
    n, c = sums.shape
    classes = W.shape[0]
    assert W.dtype == np.float32 and bias.dtype == np.float32 and W.flags.c_contiguous and W.shape == (classes, c)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    loss = C.c_float(0)
    dpooled = np.empty((n, c), dtype=np.float32)
    logits = np.empty((n, classes), dtype=np.float32)
    _L().eoq_o_head(_p(sums), C.c_int(n), C.c_int(c), C.c_int(hw), C.c_int(classes), _p(W), _p(bias), _p(labels),
                    C.c_float(lr), C.byref(loss), _p(dpooled), _p(logits))
    return float(loss.value), dpooled, logits


# --------------------------------------------------------------------------- other bit widths (Sec. 3.2.2 / 3.2.3)

def sq_int_k(a, p_a: int, k: int):
    """SQ(., k) of integer codes at exponent p_a -> (int64 codes, p_out, zero flag)."""
    a = np.ascontiguousarray(a, dtype=np.int64)
    codes = np.empty(a.shape, dtype=np.int64)
    p_out = C.c_int(0)
    z = _L().eoq_o_sq_i64_k(_p(a), C.c_size_t(a.size), C.c_int(p_a), C.c_int(k), _p(codes), C.byref(p_out))
    return codes, p_out.value, int(z)


def update_k(theta, g, p_g: int, lr_mant: int, lr_exp: int, k_u: int, k_m: int, stochastic: bool = False, seed: int = 0,
             step: int = 0, tensor_id: int = 0):
    """Update with a k_u-bit update quantizer on a k_m-bit master copy (codes at exponent -(k_m - 1)).
    -> (new master codes int32, 8-bit weight codes Q_w(master), exponent of u, zero flag)."""
    th = np.array(theta, dtype=np.int32).reshape(-1).copy()
    g = _i8(g).reshape(-1)
    assert th.size == g.size
    w8 = np.empty(th.size, dtype=np.int8)
    p_u = C.c_int(0)
    z = _L().eoq_o_update_k(_p(th), _p(w8), _p(g), C.c_int(p_g), C.c_size_t(th.size), C.c_int(lr_mant), C.c_int(lr_exp),
                            C.c_int(k_u), C.c_int(k_m), C.c_int(1 if stochastic else 0), C.c_uint64(seed), C.c_uint64(step),
                            C.c_uint64(tensor_id), C.byref(p_u))
    return th.reshape(np.shape(theta)), w8.reshape(np.shape(theta)), p_u.value, int(z)


# --------------------------------------------------------------------------- batch normalisation (comparison, Sec. 5.3)

BN_CHANNEL = np.dtype([("mu", "f8"), ("inv", "f8"), ("scale", "f4"), ("shift", "f4")])


def bn_forward(A, p: int, gamma, beta, eps: float = 1e-5):
    """Training-mode batch normalisation of a convolution output (exact integers A [n,h,w,c] at exponent p) per
    channel over the whole batch, then ReLU and Q_a2.
    -> dict(x5 int8 codes, mask 0/1, y fp32 before the ReLU, ch = per-channel constants for the backward pass)."""
    A = np.ascontiguousarray(A, dtype=np.int64)
    c = A.shape[-1]
    P = A.size // c
    gamma = np.ascontiguousarray(gamma, dtype=np.float32)
    beta = np.ascontiguousarray(beta, dtype=np.float32)
    x5 = np.empty(A.shape, dtype=np.int8)
    mask = np.empty(A.shape, dtype=np.uint8)
    y = np.empty(A.shape, dtype=np.float32)
    ch = np.zeros(c, dtype=BN_CHANNEL)
    _L().eoq_o_bn_forward(_p(A), C.c_int(p), C.c_size_t(P), C.c_int(c), _p(gamma), _p(beta), C.c_float(eps), _p(x5), _p(mask),
                          _p(y), _p(ch))
    return {"x5": x5, "mask": mask, "y": y, "ch": ch}


def bn_backward(E, p_e: int, mask01, A, p: int, gamma, ch):
    """Backward of bn_forward for error codes E at exponent p_e -> (da fp32, dgamma fp32 [c], dbeta fp32 [c])."""
    E = _i8(E)
    A = np.ascontiguousarray(A, dtype=np.int64)
    mask01 = np.ascontiguousarray(mask01, dtype=np.uint8)
    c = A.shape[-1]
    P = A.size // c
    gamma = np.ascontiguousarray(gamma, dtype=np.float32)
    da = np.empty(A.shape, dtype=np.float32)
    dgamma = np.empty(c, dtype=np.float32)
    dbeta = np.empty(c, dtype=np.float32)
    _L().eoq_o_bn_backward(_p(E), C.c_int(p_e), _p(mask01), _p(A), C.c_int(p), C.c_size_t(P), C.c_int(c), _p(gamma), _p(ch),
                           _p(da), _p(dgamma), _p(dbeta))
    return da, dgamma, dbeta

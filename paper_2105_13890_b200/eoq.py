"""Thin ctypes binding over libeoq.so (the C ABI declared in include/eoq.h).

Each function has the name and argument order of its C counterpart and only
marshals arguments: torch tensors (device memory owned by the caller) become raw
pointers, the current torch CUDA stream becomes the ``stream`` argument.  All
arithmetic runs in the CUDA kernels; there is no CPU fallback, and a missing
library raises at first use.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libeoq.so")

EOQ_OK, EOQ_ERR_BAD_ARG, EOQ_ERR_ALIGNMENT, EOQ_ERR_UNSUPPORTED, EOQ_ERR_WORKSPACE, EOQ_ERR_RANGE, EOQ_ERR_CUDA = range(7)
EOQ_DEV_TIMEOUT, EOQ_DEV_NONFINITE, EOQ_DEV_SQ_ZERO, EOQ_DEV_RANGE = 1, 2, 4, 8
EOQ_Q, EOQ_CQ, EOQ_SQ = 0, 1, 2
EOQ_ROUND_RNE, EOQ_ROUND_STOCHASTIC = 0, 1
EOQ_PASS_FWD, EOQ_PASS_DGRAD, EOQ_PASS_WGRAD = 0, 1, 2

EXPORTS = [
    "eoq_create", "eoq_destroy", "eoq_workspace_size", "eoq_conv_fwd", "eoq_conv_dgrad", "eoq_conv_wgrad",
    "eoq_quantize", "eoq_quantize_image", "eoq_err_prescale", "eoq_update", "eoq_layout_convert", "eoq_last_status",
    "eoq_last_cuda_error", "eoq_status_string", "eoq_profile_start", "eoq_profile_stop", "eoq_launch_count", "eoq_set_gemm_ctas",
    "eoq_conv_dgrad_static", "eoq_conv_fwd_dev", "eoq_weight_prep_size", "eoq_weight_prep", "eoq_conv_wgrad_dev",
    "eoq_err_prescale_dev", "eoq_update_dev", "eoq_describe_plan", "eoq_debug_force_wait_timeout", "eoq_probe_mma_i8", "eoq_profile_gemm_only", "eoq_aux_maxpool_fwd", "eoq_aux_maxpool_bwd",
    "eoq_aux_maxpool_bwd_head", "eoq_aux_avgpool_sum", "eoq_aux_join", "eoq_aux_join_head", "eoq_conv_dgrad_head", "eoq_conv_dgrad_join_head", "eoq_conv_wgrad_gemm", "eoq_wgrad_finish", "eoq_aux_head_workspace_size", "eoq_aux_head", "eoq_aux_head_update", "eoq_aux_head_error", "eoq_aux_scalar_update", "eoq_update_wide", "eoq_set_reduce_hook", "eoq_bn_workspace_size", "eoq_bn_fwd", "eoq_bn_bwd",
]
EOQ_STATIC_SCRATCH_BYTES = 16 << 20
EOQ_PROF_IGEMM_FWD, EOQ_PROF_IGEMM_DGRAD, EOQ_PROF_WGRAD = 0, 1, 2
EOQ_PROF_KINDS = 12
EOQ_PROF_NAMES = ["igemm_fwd", "igemm_dgrad", "wgrad_gemm", "err_head", "dgrad_aux", "wgrad_aux", "fwd_aux", "other", "update",
                  "input_quantizer", "wgrad_taps", "glue"]


class EoqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class eoq_conv_desc_t(C.Structure):
    _fields_ = [(k, C.c_int) for k in ("n", "h", "w", "c_in", "c_out", "kh", "kw", "stride", "pad", "x_wmargin")]

    @property
    def ho(self) -> int:
        return (self.h + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def wo(self) -> int:
        return (self.w + 2 * self.pad - self.kw) // self.stride + 1


def conv_desc(n, h, w, c_in, c_out, kh, kw, stride=1, pad=0, x_wmargin=0) -> eoq_conv_desc_t:
    return eoq_conv_desc_t(n, h, w, c_in, c_out, kh, kw, stride, pad, x_wmargin)


_lib = None
# void fn(void *user, void *device_buffer, size_t count, int dtype, int op, void *stream)
REDUCE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p, C.c_size_t, C.c_int, C.c_int, C.c_void_p)
EOQ_REDUCE_I32, EOQ_REDUCE_I64 = 0, 1
EOQ_REDUCE_MAX, EOQ_REDUCE_SUM = 0, 1


def lib() -> C.CDLL:
    """Loads libeoq.so; raises if it has not been built (python -m paper_2105_13890_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2105_13890_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, sz, u64 = C.c_void_p, C.c_int32, C.c_size_t, C.c_uint64
        dp = C.POINTER(eoq_conv_desc_t)
        L.eoq_create.argtypes = [C.POINTER(vp), C.c_int]
        L.eoq_destroy.argtypes = [vp]
        L.eoq_workspace_size.argtypes = [dp, C.c_int, C.POINTER(sz)]
        L.eoq_conv_fwd.argtypes = [vp, dp, vp, vp, i32, vp, i32, i32, vp, C.c_int, vp, vp, vp, vp, vp, sz, vp]
        L.eoq_conv_dgrad.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.eoq_conv_wgrad.argtypes = [vp, dp, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
        L.eoq_quantize.argtypes = [vp, C.c_int, vp, C.c_int, vp, sz, vp, vp, vp, sz, vp]
        L.eoq_err_prescale.argtypes = [vp, vp, vp, vp, vp, sz, i32, vp, vp, vp, vp, vp]
        L.eoq_update.argtypes = [vp, C.c_int, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(sz), i32, i32,
                                 C.c_int, u64, u64, vp]
        L.eoq_layout_convert.argtypes = [vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, vp]
        L.eoq_last_status.argtypes = [vp, vp, C.POINTER(C.c_uint)]
        L.eoq_last_cuda_error.argtypes = [vp]
        L.eoq_conv_dgrad_static.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.eoq_quantize_image.argtypes = [vp, vp] + [C.c_int] * 6 + [vp, vp, vp]
        L.eoq_profile_start.argtypes = [vp]
        L.eoq_profile_stop.argtypes = [vp, C.POINTER(C.c_int), C.POINTER(C.c_double)]
        L.eoq_launch_count.argtypes = [vp]
        L.eoq_set_gemm_ctas.argtypes = [vp, C.c_int]
        L.eoq_conv_fwd_dev.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, C.c_int, vp, vp, vp, vp]
        L.eoq_weight_prep_size.argtypes = [dp, C.POINTER(sz)]
        L.eoq_weight_prep.argtypes = [vp, C.c_int, dp, C.POINTER(vp), C.POINTER(vp), vp]
        L.eoq_conv_wgrad_dev.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.eoq_err_prescale_dev.argtypes = [vp, vp, vp, vp, vp, sz, vp, vp, vp, vp, vp, vp]
        L.eoq_update_dev.argtypes = [vp, C.c_int, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(sz), i32, i32,
                                     C.c_int, u64, vp, vp]
        L.eoq_update_wide.argtypes = [vp, C.c_int, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(sz), i32, i32,
                                      C.c_int, C.c_int, C.c_int, u64, u64, vp, vp]
        L.eoq_set_reduce_hook.argtypes = [vp, REDUCE_FN, vp]
        L.eoq_describe_plan.argtypes = [vp, dp, C.c_int, C.c_char_p, sz]
        L.eoq_debug_force_wait_timeout.argtypes = [vp]
        ci = C.c_int
        L.eoq_aux_maxpool_fwd.argtypes = [vp, vp, ci, ci, ci, ci, ci, ci, ci, vp, vp, vp]
        L.eoq_aux_maxpool_bwd.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, vp, vp, vp]
        L.eoq_aux_maxpool_bwd_head.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp]
        L.eoq_aux_avgpool_sum.argtypes = [vp, vp, ci, ci, ci, vp, vp]
        L.eoq_aux_join.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp, vp, vp, vp]
        L.eoq_conv_wgrad_gemm.argtypes = [vp, dp, vp, vp, vp, vp, sz, C.POINTER(ci), vp]
        L.eoq_wgrad_finish.argtypes = [vp, ci, dp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                       C.POINTER(vp), C.POINTER(sz), C.POINTER(ci), vp]
        L.eoq_conv_dgrad_join_head.argtypes = [vp, dp] + [vp] * 19 + [vp, sz, vp]
        L.eoq_conv_dgrad_head.argtypes = [vp, dp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.eoq_aux_join_head.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.eoq_aux_head_workspace_size.argtypes = [ci, ci, ci, C.POINTER(sz)]
        L.eoq_aux_head.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp, vp, C.c_float, vp, vp, vp, vp, sz, vp]
        L.eoq_aux_head_update.argtypes = [vp, ci, ci, ci, vp, vp, C.c_float, vp, sz, vp]
        L.eoq_aux_head_error.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp, sz, vp]
        L.eoq_aux_scalar_update.argtypes = [vp, ci, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(ci),
                                            C.POINTER(ci), C.POINTER(vp), i32, i32, ci, u64, vp, vp]
        L.eoq_bn_workspace_size.argtypes = [ci, C.POINTER(sz)]
        L.eoq_bn_fwd.argtypes = [vp, vp, ci, sz, ci, vp, vp, C.c_float, vp, vp, vp, sz, vp]
        L.eoq_bn_bwd.argtypes = [vp, vp, vp, vp, vp, ci, sz, ci, vp, vp, sz, vp, vp, vp, vp]
        L.eoq_profile_gemm_only.argtypes = [vp, C.c_int]
        L.eoq_probe_mma_i8.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double), vp]
        L.eoq_status_string.argtypes = [C.c_int]
        L.eoq_status_string.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("eoq_status_string", "eoq_launch_count"):
                getattr(L, name).restype = C.c_int
        L.eoq_launch_count.restype = C.c_ulonglong
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().eoq_status_string(int(status)).decode()


def _ptr(t) -> Optional[int]:
    """Raw address of a torch tensor (or of an int already holding one); None stays NULL."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is not None:
        return stream if isinstance(stream, int) else stream.cuda_stream
    import torch

    return torch.cuda.current_stream().cuda_stream


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def _check(status: int, where: str) -> None:
    if status != EOQ_OK:
        raise EoqError(status, where)


# ------------------------------------------------------------------------------- entry points

def eoq_create(device: int = 0) -> int:
    h = C.c_void_p()
    _check(lib().eoq_create(C.byref(h), int(device)), "eoq_create")
    return h.value


def eoq_destroy(handle: int) -> None:
    _check(lib().eoq_destroy(handle), "eoq_destroy")


def eoq_workspace_size(desc: eoq_conv_desc_t, pass_: int) -> int:
    out = C.c_size_t(0)
    _check(lib().eoq_workspace_size(C.byref(desc), int(pass_), C.byref(out)), "eoq_workspace_size")
    return out.value


def eoq_conv_fwd(handle, desc, x, x_exp, b1_c, w, gamma_c, b2_c, shortcut, relu, x5, x2=None, relu_mask=None,
                 acc_dump=None, workspace=None, stream=None, check: bool = True) -> int:
    st = lib().eoq_conv_fwd(handle, C.byref(desc), _ptr(x), _ptr(x_exp), int(b1_c), _ptr(w), int(gamma_c), int(b2_c),
                            _ptr(shortcut), 1 if relu else 0, _ptr(x5), _ptr(x2), _ptr(relu_mask), _ptr(acc_dump),
                            _ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check(st, "eoq_conv_fwd")
    return st


def eoq_conv_dgrad(handle, desc, e3, e3_exp, w, e4, e4_exp, sum_e4=None, acc_dump=None, workspace=None, stream=None,
                   check: bool = True) -> int:
    st = lib().eoq_conv_dgrad(handle, C.byref(desc), _ptr(e3), _ptr(e3_exp), _ptr(w), _ptr(e4), _ptr(e4_exp),
                              _ptr(sum_e4), _ptr(acc_dump), _ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check(st, "eoq_conv_dgrad")
    return st


def eoq_conv_wgrad(handle, desc, e3, e3_exp, x, b1_c, g, g_exp, acc_dump=None, workspace=None, stream=None,
                   check: bool = True) -> int:
    st = lib().eoq_conv_wgrad(handle, C.byref(desc), _ptr(e3), _ptr(e3_exp), _ptr(x), int(b1_c), _ptr(g), _ptr(g_exp),
                              _ptr(acc_dump), _ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check(st, "eoq_conv_wgrad")
    return st


def eoq_quantize(handle, mode, src, src_is_float, src_exp, n, dst, dst_exp=None, workspace=None, stream=None,
                 check: bool = True) -> int:
    st = lib().eoq_quantize(handle, int(mode), _ptr(src), 1 if src_is_float else 0, _ptr(src_exp), int(n), _ptr(dst),
                            _ptr(dst_exp), _ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check(st, "eoq_quantize")
    return st


def eoq_err_prescale(handle, e0, e0_exp, relu_mask, x2, n_el, gamma_c, e3, e3_exp, sum_e1=None, sum_e1x2=None,
                     stream=None, check: bool = True) -> int:
    st = lib().eoq_err_prescale(handle, _ptr(e0), _ptr(e0_exp), _ptr(relu_mask), _ptr(x2), int(n_el), int(gamma_c),
                                _ptr(e3), _ptr(e3_exp), _ptr(sum_e1), _ptr(sum_e1x2), _stream(stream))
    if check:
        _check(st, "eoq_err_prescale")
    return st


def eoq_update(handle, w: Sequence, g: Sequence, g_exp: Sequence, lr_mant: int, lr_exp: int,
               round_mode: int = EOQ_ROUND_RNE, seed: int = 0, step: int = 0, stream=None, check: bool = True) -> int:
    num = len(w)
    arr = C.c_void_p * num
    sizes = (C.c_size_t * num)(*[t.numel() for t in w])
    st = lib().eoq_update(handle, num, arr(*[_ptr(t) for t in w]), arr(*[_ptr(t) for t in g]),
                          arr(*[_ptr(t) for t in g_exp]), sizes, int(lr_mant), int(lr_exp), int(round_mode),
                          int(seed), int(step), _stream(stream))
    if check:
        _check(st, "eoq_update")
    return st


def eoq_layout_convert(handle, src, dst, n, c, h, w, to_nhwc: bool, stream=None, check: bool = True) -> int:
    st = lib().eoq_layout_convert(handle, _ptr(src), _ptr(dst), n, c, h, w, 1 if to_nhwc else 0, _stream(stream))
    if check:
        _check(st, "eoq_layout_convert")
    return st


def eoq_last_status(handle, stream=None) -> int:
    bits = C.c_uint(0)
    _check(lib().eoq_last_status(handle, _stream(stream), C.byref(bits)), "eoq_last_status")
    return bits.value


def eoq_last_cuda_error(handle) -> int:
    return lib().eoq_last_cuda_error(handle)


def eoq_quantize_image(handle, src, n, h, w, c_src, c_dst, wmargin, dst, dst_exp, stream=None, check: bool = True) -> int:
    st = lib().eoq_quantize_image(handle, _ptr(src), int(n), int(h), int(w), int(c_src), int(c_dst), int(wmargin),
                                  _ptr(dst), _ptr(dst_exp), _stream(stream))
    if check:
        _check(st, "eoq_quantize_image")
    return st


def eoq_profile_start(handle) -> None:
    _check(lib().eoq_profile_start(handle), "eoq_profile_start")


def eoq_profile_stop(handle):
    """-> ([groups per kind], [milliseconds per kind]) for the EOQ_PROF_KINDS kinds (names in EOQ_PROF_NAMES)."""
    n = (C.c_int * EOQ_PROF_KINDS)()
    ms = (C.c_double * EOQ_PROF_KINDS)()
    _check(lib().eoq_profile_stop(handle, n, ms), "eoq_profile_stop")
    return list(n), list(ms)


def eoq_set_gemm_ctas(handle, ctas: int) -> None:
    """Caps the CTAs the handle's GEMM launches use (0 = one per SM)."""
    _check(lib().eoq_set_gemm_ctas(handle, ctas), "eoq_set_gemm_ctas")


def eoq_launch_count(handle) -> int:
    return int(lib().eoq_launch_count(handle))


def eoq_conv_dgrad_static(desc, e3, e3_exp, w, e4, e4_exp, sum_e4=None, status_out=None, stream=None,
                          check: bool = True) -> int:
    """eoq_conv_dgrad for callers that may not allocate: no handle, no workspace (scratch is a static device array)."""
    st = lib().eoq_conv_dgrad_static(C.byref(desc), _ptr(e3), _ptr(e3_exp), _ptr(w), _ptr(e4), _ptr(e4_exp),
                                     _ptr(sum_e4), _ptr(status_out), _stream(stream))
    if check:
        _check(st, "eoq_conv_dgrad_static")
    return st


def eoq_conv_fwd_dev(handle, desc, x, x_exp, scalars, w, w_prep, shortcut, relu, x5, x2=None, relu_mask=None, stream=None,
                     check: bool = True) -> int:
    """eoq_conv_fwd with the scalars {b1_c, gamma_c, b2_c} in device memory and prepared weights (eoq_weight_prep)."""
    st = lib().eoq_conv_fwd_dev(handle, C.byref(desc), _ptr(x), _ptr(x_exp), _ptr(scalars), _ptr(w), _ptr(w_prep),
                                _ptr(shortcut), 1 if relu else 0, _ptr(x5), _ptr(x2), _ptr(relu_mask), _stream(stream))
    if check:
        _check(st, "eoq_conv_fwd_dev")
    return st


def eoq_weight_prep_size(desc: eoq_conv_desc_t) -> int:
    out = C.c_size_t(0)
    _check(lib().eoq_weight_prep_size(C.byref(desc), C.byref(out)), "eoq_weight_prep_size")
    return out.value


def eoq_weight_prep(handle, descs: Sequence[eoq_conv_desc_t], w: Sequence, prep: Sequence, stream=None,
                    check: bool = True) -> int:
    num = len(descs)
    darr = (eoq_conv_desc_t * num)(*descs)
    arr = C.c_void_p * num
    st = lib().eoq_weight_prep(handle, num, darr, arr(*[_ptr(t) for t in w]), arr(*[_ptr(t) for t in prep]),
                               _stream(stream))
    if check:
        _check(st, "eoq_weight_prep")
    return st


def eoq_conv_wgrad_gemm(handle, desc, e3, e3_exp, x, workspace, stream=None) -> int:
    """The weight-gradient GEMM alone; returns the slice count eoq_wgrad_finish needs for this layer."""
    parts = C.c_int(0)
    _check(lib().eoq_conv_wgrad_gemm(handle, C.byref(desc), _ptr(e3), _ptr(e3_exp), _ptr(x), _ptr(workspace), _nbytes(workspace),
                                     C.byref(parts), _stream(stream)), "eoq_conv_wgrad_gemm")
    return parts.value


def eoq_wgrad_finish(handle, descs: Sequence[eoq_conv_desc_t], e3: Sequence, e3_exp: Sequence, b1_c: Sequence, g: Sequence,
                     g_exp: Sequence, workspace: Sequence, num_parts: Sequence[int], stream=None) -> None:
    num = len(descs)
    darr = (eoq_conv_desc_t * num)(*descs)
    arr = C.c_void_p * num
    _check(lib().eoq_wgrad_finish(handle, num, darr, arr(*[_ptr(t) for t in e3]), arr(*[_ptr(t) for t in e3_exp]),
                                  arr(*[_ptr(t) for t in b1_c]), arr(*[_ptr(t) for t in g]), arr(*[_ptr(t) for t in g_exp]),
                                  arr(*[_ptr(t) for t in workspace]), (C.c_size_t * num)(*[_nbytes(t) for t in workspace]),
                                  (C.c_int * num)(*[int(v) for v in num_parts]), _stream(stream)), "eoq_wgrad_finish")


def eoq_conv_wgrad_dev(handle, desc, e3, e3_exp, x, b1_c, g, g_exp, workspace=None, stream=None, check: bool = True) -> int:
    st = lib().eoq_conv_wgrad_dev(handle, C.byref(desc), _ptr(e3), _ptr(e3_exp), _ptr(x), _ptr(b1_c), _ptr(g),
                                  _ptr(g_exp), _ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check(st, "eoq_conv_wgrad_dev")
    return st


def eoq_err_prescale_dev(handle, e0, e0_exp, relu_mask, x2, n_el, gamma_c, e3, e3_exp, sum_e1=None, sum_e1x2=None,
                         stream=None, check: bool = True) -> int:
    st = lib().eoq_err_prescale_dev(handle, _ptr(e0), _ptr(e0_exp), _ptr(relu_mask), _ptr(x2), int(n_el), _ptr(gamma_c),
                                    _ptr(e3), _ptr(e3_exp), _ptr(sum_e1), _ptr(sum_e1x2), _stream(stream))
    if check:
        _check(st, "eoq_err_prescale_dev")
    return st


def eoq_update_dev(handle, w: Sequence, g: Sequence, g_exp: Sequence, lr_mant: int, lr_exp: int, round_mode: int, seed: int,
                   step, stream=None, check: bool = True) -> int:
    """eoq_update with the step counter in device memory (a one-element int64/uint64 tensor, bumped by the call)."""
    num = len(w)
    arr = C.c_void_p * num
    sizes = (C.c_size_t * num)(*[t.numel() for t in w])
    st = lib().eoq_update_dev(handle, num, arr(*[_ptr(t) for t in w]), arr(*[_ptr(t) for t in g]),
                              arr(*[_ptr(t) for t in g_exp]), sizes, int(lr_mant), int(lr_exp), int(round_mode), int(seed),
                              _ptr(step), _stream(stream))
    if check:
        _check(st, "eoq_update_dev")
    return st


def eoq_describe_plan(handle, desc, pass_: int) -> str:
    buf = C.create_string_buffer(256)
    _check(lib().eoq_describe_plan(handle, C.byref(desc), int(pass_), buf, 256), "eoq_describe_plan")
    return buf.value.decode()


def eoq_debug_force_wait_timeout(handle) -> None:
    """Makes the next one-kernel error-head call on this handle run out at its (bounded) grid-wide wait."""
    _check(lib().eoq_debug_force_wait_timeout(handle), "eoq_debug_force_wait_timeout")


def eoq_probe_mma_i8(handle, n_cols: int, iters: int, launches: int, stream=None):
    """-> (TOPS over the timed launches, SM cycles per 128 x n_cols x 32 MMA) of tcgen05.mma kind::i8."""
    tops, cyc = C.c_double(0), C.c_double(0)
    _check(lib().eoq_probe_mma_i8(handle, int(n_cols), int(iters), int(launches), C.byref(tops), C.byref(cyc), _stream(stream)),
           "eoq_probe_mma_i8")
    return tops.value, cyc.value


def eoq_profile_gemm_only(handle, on: bool) -> None:
    """Timing aid: dgrad / wgrad calls launch their GEMM kernel only (their outputs are then not produced)."""
    _check(lib().eoq_profile_gemm_only(handle, 1 if on else 0), "eoq_profile_gemm_only")


# ------------------------------------------------------------------------------- network glue

def eoq_aux_maxpool_fwd(handle, x, n, h, w, c, k, stride, pad, y, arg, stream=None) -> None:
    _check(lib().eoq_aux_maxpool_fwd(handle, _ptr(x), n, h, w, c, k, stride, pad, _ptr(y), _ptr(arg), _stream(stream)),
           "eoq_aux_maxpool_fwd")


def eoq_aux_maxpool_bwd(handle, e, e_exp, arg, n, h, w, c, k, stride, pad, e_in, e_in_exp, stream=None) -> None:
    _check(lib().eoq_aux_maxpool_bwd(handle, _ptr(e), _ptr(e_exp), _ptr(arg), n, h, w, c, k, stride, pad, _ptr(e_in),
                                     _ptr(e_in_exp), _stream(stream)), "eoq_aux_maxpool_bwd")


def eoq_aux_maxpool_bwd_head(handle, e, e_exp, arg, n, h, w, c, k, stride, pad, e_in, e_in_exp, relu_mask, gamma, e3, e3_exp,
                             sum_e1=None, stream=None) -> None:
    _check(lib().eoq_aux_maxpool_bwd_head(handle, _ptr(e), _ptr(e_exp), _ptr(arg), n, h, w, c, k, stride, pad, _ptr(e_in),
                                          _ptr(e_in_exp), _ptr(relu_mask), _ptr(gamma), _ptr(e3), _ptr(e3_exp), _ptr(sum_e1),
                                          _stream(stream)), "eoq_aux_maxpool_bwd_head")


def eoq_bn_workspace_size(c) -> int:
    out = C.c_size_t(0)
    _check(lib().eoq_bn_workspace_size(c, C.byref(out)), "eoq_bn_workspace_size")
    return out.value


def eoq_bn_fwd(handle, acc, acc_exp, pixels, c, gamma, beta, eps, x5, relu_mask, workspace, stream=None) -> None:
    _check(lib().eoq_bn_fwd(handle, _ptr(acc), acc_exp, int(pixels), c, _ptr(gamma), _ptr(beta), eps, _ptr(x5), _ptr(relu_mask),
                            _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)), "eoq_bn_fwd")


def eoq_bn_bwd(handle, e, e_exp, relu_mask, acc, acc_exp, pixels, c, gamma, workspace, da, dgamma, dbeta, stream=None) -> None:
    _check(lib().eoq_bn_bwd(handle, _ptr(e), _ptr(e_exp), _ptr(relu_mask), _ptr(acc), acc_exp, int(pixels), c, _ptr(gamma),
                            _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(da), _ptr(dgamma), _ptr(dbeta),
                            _stream(stream)), "eoq_bn_bwd")


def eoq_aux_avgpool_sum(handle, x, n, hw, c, sums, stream=None) -> None:
    _check(lib().eoq_aux_avgpool_sum(handle, _ptr(x), n, hw, c, _ptr(sums), _stream(stream)), "eoq_aux_avgpool_sum")


def eoq_aux_join(handle, a, a_exp, b, b_exp, mask_b, n_el, out, out_exp, sum_out=None, stream=None) -> None:
    _check(lib().eoq_aux_join(handle, _ptr(a), _ptr(a_exp), _ptr(b), _ptr(b_exp), _ptr(mask_b), int(n_el), _ptr(out),
                              _ptr(out_exp), _ptr(sum_out), _stream(stream)), "eoq_aux_join")


def eoq_conv_dgrad_join_head(handle, desc, e3, e3_exp, w, e4, e4_exp, sum_e4, b, b_exp, mask_b, out, out_exp, sum_out, next_mask=None,
                             next_x2=None, next_gamma=None, next_e3=None, next_e3_exp=None, next_sum_e1=None, next_sum_e1x2=None,
                             workspace=None, stream=None) -> None:
    _check(lib().eoq_conv_dgrad_join_head(handle, C.byref(desc), _ptr(e3), _ptr(e3_exp), _ptr(w), _ptr(e4), _ptr(e4_exp), _ptr(sum_e4),
                                          _ptr(b), _ptr(b_exp), _ptr(mask_b), _ptr(out), _ptr(out_exp), _ptr(sum_out), _ptr(next_mask),
                                          _ptr(next_x2), _ptr(next_gamma), _ptr(next_e3), _ptr(next_e3_exp), _ptr(next_sum_e1),
                                          _ptr(next_sum_e1x2), _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "eoq_conv_dgrad_join_head")


def eoq_conv_dgrad_head(handle, desc, e3, e3_exp, w, e4, e4_exp, sum_e4, next_mask, next_x2, next_gamma, next_e3, next_e3_exp,
                        next_sum_e1=None, next_sum_e1x2=None, workspace=None, stream=None) -> None:
    _check(lib().eoq_conv_dgrad_head(handle, C.byref(desc), _ptr(e3), _ptr(e3_exp), _ptr(w), _ptr(e4), _ptr(e4_exp), _ptr(sum_e4),
                                     _ptr(next_mask), _ptr(next_x2), _ptr(next_gamma), _ptr(next_e3), _ptr(next_e3_exp),
                                     _ptr(next_sum_e1), _ptr(next_sum_e1x2), _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "eoq_conv_dgrad_head")


def eoq_aux_join_head(handle, a, a_exp, b, b_exp, mask_b, n_el, out, out_exp, sum_out, relu_mask, x2, gamma, e3, e3_exp, sum_e1=None,
                      sum_e1x2=None, stream=None) -> None:
    _check(lib().eoq_aux_join_head(handle, _ptr(a), _ptr(a_exp), _ptr(b), _ptr(b_exp), _ptr(mask_b), int(n_el), _ptr(out), _ptr(out_exp),
                                   _ptr(sum_out), _ptr(relu_mask), _ptr(x2), _ptr(gamma), _ptr(e3), _ptr(e3_exp), _ptr(sum_e1),
                                   _ptr(sum_e1x2), _stream(stream)), "eoq_aux_join_head")


def eoq_aux_head_workspace_size(n, c, classes) -> int:
    out = C.c_size_t(0)
    _check(lib().eoq_aux_head_workspace_size(n, c, classes, C.byref(out)), "eoq_aux_head_workspace_size")
    return out.value


def eoq_aux_head(handle, sums, n, c, hw, classes, W, bias, labels, lr, loss, dpooled, logits, workspace, stream=None) -> None:
    _check(lib().eoq_aux_head(handle, _ptr(sums), n, c, hw, classes, _ptr(W), _ptr(bias), _ptr(labels), float(lr), _ptr(loss),
                              _ptr(dpooled), _ptr(logits), _ptr(workspace), _nbytes(workspace), _stream(stream)), "eoq_aux_head")


def eoq_aux_head_update(handle, n, c, classes, W, bias, lr, workspace, stream=None) -> None:
    _check(lib().eoq_aux_head_update(handle, n, c, classes, _ptr(W), _ptr(bias), lr, _ptr(workspace), _nbytes(workspace),
                                     _stream(stream)), "eoq_aux_head_update")


def eoq_aux_head_error(handle, dpooled, n, c, hw, e, e_exp, workspace, stream=None) -> None:
    _check(lib().eoq_aux_head_error(handle, _ptr(dpooled), n, c, hw, _ptr(e), _ptr(e_exp), _ptr(workspace), _nbytes(workspace),
                                    _stream(stream)), "eoq_aux_head_error")


def eoq_aux_scalar_update(handle, theta: Sequence, mirror: Sequence, total: Sequence, total_exp: Sequence, exp_bias: Sequence[int],
                          tensor_id: Sequence[int], grad_out: Sequence, lr_mant: int, lr_exp: int, round_mode: int, seed: int,
                          step=None, stream=None) -> None:
    num = len(theta)
    arr = C.c_void_p * num
    iarr = C.c_int * num
    _check(lib().eoq_aux_scalar_update(handle, num, arr(*[_ptr(t) for t in theta]), arr(*[_ptr(t) for t in mirror]),
                                       arr(*[_ptr(t) for t in total]), arr(*[_ptr(t) for t in total_exp]), iarr(*exp_bias),
                                       iarr(*tensor_id), arr(*[_ptr(t) for t in grad_out]), int(lr_mant), int(lr_exp),
                                       int(round_mode), int(seed), _ptr(step), _stream(stream)), "eoq_aux_scalar_update")


def eoq_update_wide(handle, master: Sequence, w: Sequence, g: Sequence, g_exp: Sequence, lr_mant: int, lr_exp: int, k_u: int,
                    k_m: int, round_mode: int = EOQ_ROUND_RNE, seed: int = 0, step: int = 0, step_dev=None, stream=None) -> None:
    """The update with a k_u-bit update quantizer on k_m-bit master codes (int32 tensors); w receives Q_w(master)."""
    num = len(w)
    arr = C.c_void_p * num
    sizes = (C.c_size_t * num)(*[t.numel() for t in w])
    _check(lib().eoq_update_wide(handle, num, arr(*[_ptr(t) for t in master]), arr(*[_ptr(t) for t in w]),
                                 arr(*[_ptr(t) for t in g]), arr(*[_ptr(t) for t in g_exp]), sizes, int(lr_mant), int(lr_exp),
                                 int(k_u), int(k_m), int(round_mode), int(seed), int(step), _ptr(step_dev), _stream(stream)),
           "eoq_update_wide")


def eoq_set_reduce_hook(handle, fn) -> None:
    """Installs (fn = a REDUCE_FN instance, which the caller keeps alive) or removes (fn = None) the all-reduce hook of
    a handle: see eoq_set_reduce_hook in eoq.h."""
    _check(lib().eoq_set_reduce_hook(handle, fn if fn is not None else REDUCE_FN(), None), "eoq_set_reduce_hook")

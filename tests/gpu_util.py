"""Helpers for the GPU parity tests: device buffers, one shared handle, comparisons against the oracle."""
import numpy as np
import torch

from paper_2105_13890_b200 import eoq

_handle = None


def handle():
    global _handle
    if _handle is None:
        _handle = eoq.eoq_create(0)
    return _handle


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0")


def empty(shape, dtype):
    return torch.empty(shape, dtype=dtype, device="cuda:0")


def zeros(shape, dtype):
    return torch.zeros(shape, dtype=dtype, device="cuda:0")


def workspace(desc, pass_):
    n = max(eoq.eoq_workspace_size(desc, pass_), 256)
    return torch.empty(n, dtype=torch.uint8, device="cuda:0")


def gdesc(d):
    return eoq.conv_desc(d.n, d.h, d.w, d.c_in, d.c_out, d.kh, d.kw, d.stride, d.pad)


def host(t):
    return t.cpu().numpy()


def unpack_mask(mask_t, shape):
    return np.unpackbits(host(mask_t), bitorder="little")[: int(np.prod(shape))].reshape(shape)


def pack_mask(mask01):
    return np.packbits(np.ascontiguousarray(mask01, dtype=np.uint8).reshape(-1), bitorder="little")


def status_clear():
    return eoq.eoq_last_status(handle())

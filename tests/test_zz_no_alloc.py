"""The allocation-free dgrad entry point against the regular one.

eoq_conv_dgrad_static serves callers that may not allocate device memory (no handle, no workspace: its scratch
is a static device array inside the library).  It must give the same e4 codes, exponent and code sum as
eoq_conv_dgrad and as the oracle, on a first call and again on a second call that finds the array dirty from the first.
Collected last on purpose: if it fails, every other test has already run.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import ConvDesc
from paper_2105_13890_b200 import eoq, synth

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0")


def _zeros(shape, dt):
    return torch.zeros(shape, dtype=dt, device="cuda:0")


def _case(n, h, w, c_in, c_out, k, stride, pad, seed):
    ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
    e3 = synth.normal_codes((n, ho, wo, c_out), seed, 0)
    wt = synth.int8_uniform((c_out, k, k, c_in), seed, 1, -25, 25)
    return eoq.conv_desc(n, h, w, c_in, c_out, k, k, stride, pad), e3, wt


def test_static_dgrad_matches_regular_entry_point_twice_in_a_row():
    handle = eoq.eoq_create(0)
    try:
        cases = [_case(8, 32, 32, 16, 16, 3, 1, 1, 901), _case(2, 28, 28, 64, 128, 3, 2, 1, 902)]
        for call, (desc, e3, wt) in enumerate(cases + cases[:1]):  # third call repeats the first geometry
            shape = (desc.n, desc.h, desc.w, desc.c_in)
            e3_d, w_d, p3 = _dev(e3), _dev(wt), _dev(np.array([-10 - call], dtype=np.int32))
            ws = torch.empty(eoq.eoq_workspace_size(desc, eoq.EOQ_PASS_DGRAD), dtype=torch.uint8, device="cuda:0")
            ref_e4, ref_exp, ref_sum = _zeros(shape, torch.int8), _zeros(1, torch.int32), _zeros(1, torch.int64)
            eoq.eoq_conv_dgrad(handle, desc, e3_d, p3, w_d, ref_e4, ref_exp, ref_sum, None, ws)
            assert eoq.eoq_last_status(handle) == 0
            got_e4, got_exp, got_sum = _zeros(shape, torch.int8), _zeros(1, torch.int32), _zeros(1, torch.int64)
            status = torch.full((1,), 99, dtype=torch.int32, device="cuda:0")
            eoq.eoq_conv_dgrad_static(desc, e3_d, p3, w_d, got_e4, got_exp, got_sum, status)
            torch.cuda.synchronize()
            assert status.item() == 0
            assert torch.equal(got_e4, ref_e4)          # integer codes: bit for bit
            assert got_exp.item() == ref_exp.item() and got_sum.item() == ref_sum.item()
            assert got_e4.any()
            # and against the oracle itself
            od = ConvDesc(desc.n, desc.h, desc.w, desc.c_in, desc.c_out, desc.kh, desc.kw, desc.stride, desc.pad)
            want, p4, _ = oracle.sq_int(oracle.conv_dgrad_acc(od, e3, wt), -10 - call - 7)
            assert np.array_equal(got_e4.cpu().numpy().astype(np.int32), want) and got_exp.item() == p4
            assert got_sum.item() == int(want.astype(np.int64).sum())
    finally:
        eoq.eoq_destroy(handle)


def test_static_dgrad_rejects_geometry_beyond_its_scratch():
    desc, e3, wt = _case(64, 56, 56, 64, 64, 3, 1, 1, 903)  # 51 MB of int32 sums: more than the static array
    assert eoq.eoq_workspace_size(desc, eoq.EOQ_PASS_DGRAD) > eoq.EOQ_STATIC_SCRATCH_BYTES
    tiny = _zeros(16, torch.int8)
    st = eoq.eoq_conv_dgrad_static(desc, tiny, _zeros(1, torch.int32), tiny, tiny, _zeros(1, torch.int32), check=False)
    assert st == eoq.EOQ_ERR_WORKSPACE

"""Data-parallel replicas through the library's all-reduce hook, emulated on one GPU without any kernel waiting for
another: each of two replicas (half of the batch each) first runs with a hook that only records the local values it
would exchange; the recorded values are combined on the host side of the test (maximum or sum, as the hook's
operation says); then each replica runs again with a hook that writes the combined value into the buffer, which is
exactly what an all-reduce leaves there.  Activations and errors of the two replicas, concatenated, and the weight
gradient of either must equal, bit for bit, what one device computes on the whole batch (and the oracle)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import ConvDesc
from paper_2105_13890_b200 import eoq, ranks, synth

import gpu_util as G

pytestmark = pytest.mark.gpu


class Recorder:
    def __init__(self):
        self.log = []
        self.fn = eoq.REDUCE_FN(self._call)

    def _call(self, user, ptr, count, dtype, op, stream):
        self.log.append((op, ranks.device_tensor(ptr, count, dtype).clone()))   # stream-ordered copy of the local value


class Injector:
    def __init__(self, values):
        self.values, self.i = values, 0
        self.fn = eoq.REDUCE_FN(self._call)

    def _call(self, user, ptr, count, dtype, op, stream):
        ranks.device_tensor(ptr, count, dtype).copy_(self.values[self.i])      # what an all-reduce would leave
        self.i += 1


def run_layer(h, d, x0, w, e0, p0, scal):
    """Forward, error head, dgrad and wgrad of one layer on handle h."""
    gd = G.gdesc(d)
    shape = (d.n, d.ho, d.wo, d.c_out)
    n_out = int(np.prod(shape))
    b1, gamma, b2 = scal
    x_d, w_d = G.dev(x0), G.dev(w)
    x5, x2 = G.zeros(shape, torch.int8), G.zeros(shape, torch.int16)
    mask = G.zeros((n_out + 7) // 8, torch.uint8)
    eoq.eoq_conv_fwd(h, gd, x_d, None, b1, w_d, gamma, b2, None, True, x5, x2, mask, None, G.workspace(gd, eoq.EOQ_PASS_FWD))
    e3, e3_exp = G.zeros(shape, torch.int8), G.zeros(1, torch.int32)
    s1, s2 = G.zeros(1, torch.int64), G.zeros(1, torch.int64)
    eoq.eoq_err_prescale(h, G.dev(e0), G.dev(np.array([p0], dtype=np.int32)), mask, x2, n_out, gamma, e3, e3_exp, s1, s2)
    e4, e4_exp, s4 = G.zeros(x0.shape, torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
    eoq.eoq_conv_dgrad(h, gd, e3, e3_exp, w_d, e4, e4_exp, s4, None, G.workspace(gd, eoq.EOQ_PASS_DGRAD))
    g, g_exp = G.zeros(w.shape, torch.int8), G.zeros(1, torch.int32)
    eoq.eoq_conv_wgrad(h, gd, e3, e3_exp, x_d, b1, g, g_exp, None, G.workspace(gd, eoq.EOQ_PASS_WGRAD))
    out = {"x5": x5, "e3": e3, "p3": e3_exp, "e4": e4, "p4": e4_exp, "g": g, "pg": g_exp, "s1": s1, "s2": s2, "s4": s4}
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("d", [ConvDesc(4, 12, 12, 64, 64, 3, 3, 1, 1), ConvDesc(4, 16, 16, 32, 64, 3, 3, 2, 1),
                               ConvDesc(6, 9, 9, 64, 128, 1, 1, 1, 0)], ids=["3x3", "3x3_stride2", "1x1"])
def test_two_replicas_through_the_reduce_hook_equal_one_device(d):
    x0 = synth.relu_codes((d.n, d.h, d.w, d.c_in), 9000 + d.c_in, 0)
    w = synth.int8_uniform((d.c_out, d.kh, d.kw, d.c_in), 9001, 1, -20, 20)
    e0 = synth.normal_codes((d.n, d.ho, d.wo, d.c_out), 9002, 2)
    scal, p0 = (-2, 118, 3), -12
    h = eoq.eoq_create(0)
    try:
        whole = run_layer(h, d, x0, w, e0, p0, scal)
        half = ConvDesc(d.n // 2, d.h, d.w, d.c_in, d.c_out, d.kh, d.kw, d.stride, d.pad)
        parts = [slice(0, d.n // 2), slice(d.n // 2, d.n)]
        logs = []
        for sl in parts:                                   # pass 1: what would each replica send?
            rec = Recorder()
            eoq.eoq_set_reduce_hook(h, rec.fn)
            run_layer(h, half, x0[sl], w, e0[sl], p0, scal)
            assert eoq.eoq_last_status(h) == 0
            logs.append(rec.log)
        assert len(logs[0]) == len(logs[1]) > 0
        combined = []
        for (op, a), (op_b, b) in zip(*logs):
            assert op == op_b
            combined.append(torch.maximum(a, b) if op == eoq.EOQ_REDUCE_MAX else a + b)
        reps = []
        for sl in parts:                                   # pass 2: every exchange returns the combined value
            inj = Injector(combined)
            eoq.eoq_set_reduce_hook(h, inj.fn)
            reps.append(run_layer(h, half, x0[sl], w, e0[sl], p0, scal))
            assert inj.i == len(combined) and eoq.eoq_last_status(h) == 0
        eoq.eoq_set_reduce_hook(h, None)
        for key in ("x5", "e3", "e4"):
            assert torch.equal(torch.cat([reps[0][key], reps[1][key]]), whole[key]), key
        for r in reps:
            for key in ("p3", "p4", "g", "pg", "s1", "s2", "s4"):
                assert torch.equal(r[key], whole[key]), key
        # and the whole-batch run is the oracle's
        fwd = oracle.layer_forward(d, x0, scal[0], w, scal[1], scal[2])
        bwd = oracle.layer_backward(d, e0, p0, fwd["mask"], fwd["x2"], x0, scal[0], w, scal[1])
        assert np.array_equal(G.host(whole["e4"]), bwd["e4"]) and np.array_equal(G.host(whole["g"]), bwd["g_w"])
    finally:
        eoq.eoq_destroy(h)


def test_join_pooling_and_input_quantizer_through_the_hook():
    """The glue calls that reduce over the batch (error join, max-pool backward, input quantizer) split over two
    replicas the same way."""
    h = eoq.eoq_create(0)
    try:
        n, hh, ww, c = 4, 10, 10, 32
        a = synth.normal_codes((n, hh, ww, c), 9200, 0)
        b = synth.normal_codes((n, hh, ww, c), 9200, 1)
        x = synth.relu_codes((n, hh, ww, c), 9200, 2)
        e = synth.normal_codes((n, 5, 5, c), 9200, 3)
        img = synth.normal_f32((n, 12, 12, 3), 9200, 4)
        m01 = synth.bits((n, hh, ww, c), 9200, 5, 0.5)
        x2 = (synth.relu_codes((n, hh, ww, c), 9200, 6).astype(np.int32) * 31).astype(np.int16)
        gam = G.dev(np.array([109], dtype=np.int32))

        def run(sl):
            m = sl.stop - sl.start
            out = {}
            j, pj, sj = G.zeros((m, hh, ww, c), torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
            eoq.eoq_aux_join(h, G.dev(a[sl]), G.dev(np.array([-11], dtype=np.int32)), G.dev(b[sl]), G.dev(np.array([-14], dtype=np.int32)),
                             None, j.numel(), j, pj, sj)
            y, arg = G.zeros((m, 5, 5, c), torch.int8), G.zeros((m, 5, 5, c), torch.uint8)
            eoq.eoq_aux_maxpool_fwd(h, G.dev(x[sl]), m, hh, ww, c, 3, 2, 1, y, arg)
            ein, pin = G.zeros((m, hh, ww, c), torch.int8), G.zeros(1, torch.int32)
            eoq.eoq_aux_maxpool_bwd(h, G.dev(e[sl]), G.dev(np.array([-13], dtype=np.int32)), arg, m, hh, ww, c, 3, 2, 1, ein, pin)
            q, pq = G.zeros((m, 12, 12, 16), torch.int8), G.zeros(1, torch.int32)
            eoq.eoq_quantize_image(h, G.dev(img[sl]), m, 12, 12, 3, 16, 0, q, pq)
            # the same producers with their consumer's error head fused in: two maxima and up to three sums to exchange
            mk, x2d = G.dev(G.pack_mask(m01[sl])), G.dev(x2[sl])
            j2, pj2, sj2 = G.zeros((m, hh, ww, c), torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
            h3, ph3, hs1, hs2 = G.zeros((m, hh, ww, c), torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64), G.zeros(1, torch.int64)
            eoq.eoq_aux_join_head(h, G.dev(a[sl]), G.dev(np.array([-11], dtype=np.int32)), G.dev(b[sl]), G.dev(np.array([-14], dtype=np.int32)),
                                  None, j2.numel(), j2, pj2, sj2, mk, x2d, gam, h3, ph3, hs1, hs2)
            ein2, pin2 = G.zeros((m, hh, ww, c), torch.int8), G.zeros(1, torch.int32)
            p3, pp3, ps1 = G.zeros((m, hh, ww, c), torch.int8), G.zeros(1, torch.int32), G.zeros(1, torch.int64)
            eoq.eoq_aux_maxpool_bwd_head(h, G.dev(e[sl]), G.dev(np.array([-13], dtype=np.int32)), arg, m, hh, ww, c, 3, 2, 1, ein2, pin2, mk,
                                         gam, p3, pp3, ps1)
            torch.cuda.synchronize()
            return {"j": j, "pj": pj, "sj": sj, "ein": ein, "pin": pin, "q": q, "pq": pq, "j2": j2, "pj2": pj2, "sj2": sj2, "h3": h3,
                    "ph3": ph3, "hs1": hs1, "hs2": hs2, "ein2": ein2, "pin2": pin2, "p3": p3, "pp3": pp3, "ps1": ps1}

        whole = run(slice(0, n))
        parts = [slice(0, 2), slice(2, 4)]
        logs = []
        for sl in parts:
            rec = Recorder()
            eoq.eoq_set_reduce_hook(h, rec.fn)
            run(sl)
            logs.append(rec.log)
        combined = [torch.maximum(x1, x2) if op == eoq.EOQ_REDUCE_MAX else x1 + x2 for (op, x1), (_, x2) in zip(*logs)]
        reps = []
        for sl in parts:
            inj = Injector(combined)
            eoq.eoq_set_reduce_hook(h, inj.fn)
            reps.append(run(sl))
        eoq.eoq_set_reduce_hook(h, None)
        for key in ("j", "ein", "q", "j2", "h3", "ein2", "p3"):
            assert torch.equal(torch.cat([reps[0][key], reps[1][key]]), whole[key]), key
        for r in reps:
            for key in ("pj", "sj", "pin", "pq", "pj2", "sj2", "ph3", "hs1", "hs2", "pin2", "pp3", "ps1"):
                assert torch.equal(r[key], whole[key]), key
        assert torch.equal(whole["j2"], whole["j"]) and torch.equal(whole["ein2"], whole["ein"])
        S, p = oracle.join(a, -11, b, -14)
        ref, pr, _ = oracle.sq_int(S, p)
        assert np.array_equal(G.host(whole["j"]).astype(np.int32), ref) and whole["pj"].item() == pr
    finally:
        eoq.eoq_destroy(h)

"""A whole step over a small network: the graph replay with the weight-gradient chain on a side stream must leave
exactly what the call-by-call step on one stream leaves (same kernels, different scheduling), and the first layer's
results must match the oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import ConvDesc
from paper_2105_13890_b200 import eoq, synth, workloads
from paper_2105_13890_b200.step import Scalars, TrainStep

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,batch", [("resnet20", 4), ("resnet18", 1)])
def test_graph_replay_equals_eager_step(name, batch):
    wl = workloads.get(name, batch)
    h1, h2 = eoq.eoq_create(0), eoq.eoq_create(0)
    a = TrainStep(wl, h1, scalars=Scalars())
    b = TrainStep(wl, h2, scalars=Scalars())
    a.run()
    torch.cuda.synchronize()
    assert a.status() & eoq.EOQ_DEV_TIMEOUT == 0
    # the capture runs the step twice (warm-up + capture): restore the weights b started from before replaying
    w0 = [lb.w.clone() for lb in b.layers]
    b.capture(overlap=True)
    for lb, w in zip(b.layers, w0):
        lb.w.copy_(w)
    b.step_no = 0
    b.replay()
    torch.cuda.synchronize()
    assert b.status() & eoq.EOQ_DEV_TIMEOUT == 0
    # the captured update carries step counter 1 (second run), the eager one 0: compare everything but the weights
    for la, lb in zip(a.layers, b.layers):
        for key in ("x5", "e3", "e3_exp", "g", "g_exp"):
            assert torch.equal(getattr(la, key), getattr(lb, key)), (la.layer.name, key)
        if la.e4 is not None:
            assert torch.equal(la.e4, lb.e4) and torch.equal(la.e4_exp, lb.e4_exp), la.layer.name
    assert any(not torch.equal(la.w, w) for la, w in zip(a.layers, w0))  # the update moved weights


def test_first_layer_of_a_step_matches_the_oracle():
    wl = workloads.get("resnet20", 2)
    st = TrainStep(wl, eoq.eoq_create(0), scalars=Scalars())
    w_before = st.layers[1].w.clone()
    st.run()
    torch.cuda.synchronize()
    l = wl.layers[1]
    lb = st.layers[1]
    d = ConvDesc(l.n, l.h, l.w, l.c_in, l.c_out, l.k, l.k, l.stride, l.pad)
    x0 = lb.x0.cpu().numpy()
    fwd = oracle.layer_forward(d, x0, st.sc.b1_c, w_before.cpu().numpy(), 128, st.sc.b2_c)
    assert np.array_equal(lb.x5.cpu().numpy(), fwd["x5"])
    bwd = oracle.layer_backward(d, lb.e0.cpu().numpy(), -12, fwd["mask"], None, x0, st.sc.b1_c, w_before.cpu().numpy(), 128)
    assert np.array_equal(lb.e3.cpu().numpy(), bwd["e3"]) and lb.e3_exp.item() == bwd["p3"]
    assert np.array_equal(lb.e4.cpu().numpy(), bwd["e4"]) and lb.e4_exp.item() == bwd["p4"]
    assert np.array_equal(lb.g.cpu().numpy(), bwd["g_w"]) and lb.g_exp.item() == bwd["p_gw"]
    want, _, _ = oracle.update(w_before.cpu().numpy(), bwd["g_w"], bwd["p_gw"], st.lr_mant, st.lr_exp, stochastic=True,
                               seed=synth.BASE_SEED, step=0, tensor_id=1)
    assert np.array_equal(lb.w.cpu().numpy().astype(np.int32), want)

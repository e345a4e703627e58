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


def _host_inputs(st, wl):
    """The step's inputs regenerated on the host from the seeded streams (what TrainStep uploaded), with the
    weights quantized by the oracle."""
    seed = synth.BASE_SEED
    out = []
    pools = {}

    def pooled(kind, shape, stream):
        # TrainStep draws one tensor per (kind, shape) and reuses it for every buffer of that kind and shape
        if (kind, shape) not in pools:
            pools[(kind, shape)] = (synth.relu_codes if kind == "relu" else synth.normal_codes)(shape, seed, stream)
        return pools[(kind, shape)]

    for i, l in enumerate(wl.layers):
        x0 = None if i == 0 else pooled("relu", (l.n, l.h, l.w, l.c_in), 1)
        e0 = pooled("err", (l.n, l.ho, l.wo, l.c_out), 2)
        sc = pooled("relu", (l.n, l.ho, l.wo, l.c_out), 3) if l.shortcut else None
        wf = workloads.init_weight_f32(l, wl, synth.normal_f64((l.c_out, l.k, l.k, l.c_in), seed, 100 + i))
        out.append((x0, e0, sc, oracle.q_w(wf)))
    return out


@pytest.mark.parametrize("name,batch", [("resnet20", 2), ("resnet110", 1), ("resnet18", 1), ("resnet34", 1), ("resnet50", 1)])
def test_every_layer_of_a_step_matches_the_oracle(name, batch):
    """One whole step of each network at a small batch: every layer's activation, error, weight gradient
    (codes and exponents), reduction sums and updated weights against the oracle, which is fed the same seeded
    inputs generated on the host."""
    wl = workloads.get(name, batch)
    st = TrainStep(wl, eoq.eoq_create(0), scalars=Scalars())
    host = _host_inputs(st, wl)
    for lb, (_, _, _, wq) in zip(st.layers, host):
        assert np.array_equal(lb.w.cpu().numpy(), wq), lb.layer.name   # Q_w at initialisation
    st.run()
    torch.cuda.synchronize()
    assert st.status() & eoq.EOQ_DEV_TIMEOUT == 0
    sc = st.sc
    for i, (lb, (x0, e0, short, wq)) in enumerate(zip(st.layers, host)):
        l = lb.layer
        d = ConvDesc(l.n, l.h, l.w, l.c_in, l.c_out, l.k, l.k, l.stride, l.pad)
        gamma = sc.gamma_c if l.gamma_trainable else 128
        b1 = 0 if i == 0 else sc.b1_c
        x_exp = -7
        if i == 0:
            # the network input: SQ of the fp32 image padded to the stored channel count
            img = st.host_image(synth.BASE_SEED)
            padded = np.zeros(img.shape[:3] + (l.c_in,), dtype=np.float32)
            padded[..., :img.shape[3]] = img
            codes, x_exp, _ = oracle.quantize_f32(oracle.MODE_SQ, padded)
            x0 = codes.astype(np.int8)
            m = lb.wmargin
            stored = lb.x0.cpu().numpy()
            assert np.array_equal(stored[:, :, m:m + l.w, :], x0) and st.image_exp.item() == x_exp
        fwd = oracle.layer_forward(d, x0, b1, wq, gamma, sc.b2_c if l.relu else 0, short, l.relu, x_exp=x_exp)
        assert np.array_equal(lb.x5.cpu().numpy(), fwd["x5"]), (l.name, "x5")
        if lb.x2 is not None:
            assert np.array_equal(lb.x2.cpu().numpy().astype(np.int32), fwd["x2"]), (l.name, "x2")
        bwd = oracle.layer_backward(d, e0, -12, fwd["mask"] if l.relu else np.ones_like(fwd["mask"]),
                                    fwd["x2"] if lb.x2 is not None else None, x0, b1, wq, gamma)
        assert np.array_equal(lb.e3.cpu().numpy(), bwd["e3"]) and lb.e3_exp.item() == bwd["p3"], (l.name, "e3")
        assert lb.sum_e1.item() == bwd["sum_e1"], (l.name, "sum_e1")
        if lb.x2 is not None:
            assert lb.sum_e1x2.item() == bwd["sum_e1x2"], (l.name, "sum_e1x2")
        if l.has_dgrad:
            assert np.array_equal(lb.e4.cpu().numpy(), bwd["e4"]) and lb.e4_exp.item() == bwd["p4"], (l.name, "e4")
            assert lb.sum_e4.item() == bwd["sum_e4"], (l.name, "sum_e4")
        assert np.array_equal(lb.g.cpu().numpy(), bwd["g_w"]) and lb.g_exp.item() == bwd["p_gw"], (l.name, "g_w")
        want, _, _ = oracle.update(wq, bwd["g_w"], bwd["p_gw"], st.lr_mant, st.lr_exp, stochastic=True,
                                   seed=synth.BASE_SEED, step=0, tensor_id=i)
        assert np.array_equal(lb.w.cpu().numpy().astype(np.int32), want), (l.name, "w")


@pytest.mark.parametrize("batch", [1, 2, 4])
def test_weight_trajectory_over_consecutive_steps(batch):
    """Small-batch online training: several consecutive steps (each with its own stochastic-rounding draws) must
    leave, after every step, exactly the int8 weights the oracle reaches when it repeats the same steps."""
    steps = 4
    wl = workloads.get("resnet20", batch)
    st = TrainStep(wl, eoq.eoq_create(0), scalars=Scalars(), lr_mant=3, lr_exp=-4)
    host = _host_inputs(st, wl)
    sc = st.sc
    w_ref = [wq.copy() for (_, _, _, wq) in host]
    img = st.host_image(synth.BASE_SEED)
    changed = 0
    for k in range(steps):
        st.run()
        torch.cuda.synchronize()
        assert st.status() & eoq.EOQ_DEV_TIMEOUT == 0
        for i, (lb, (x0, e0, short, _)) in enumerate(zip(st.layers, host)):
            l = lb.layer
            d = ConvDesc(l.n, l.h, l.w, l.c_in, l.c_out, l.k, l.k, l.stride, l.pad)
            gamma = sc.gamma_c if l.gamma_trainable else 128
            b1 = 0 if i == 0 else sc.b1_c
            x_exp = -7
            if i == 0:
                padded = np.zeros(img.shape[:3] + (l.c_in,), dtype=np.float32)
                padded[..., :img.shape[3]] = img
                codes, x_exp, _ = oracle.quantize_f32(oracle.MODE_SQ, padded)
                x0 = codes.astype(np.int8)
            fwd = oracle.layer_forward(d, x0, b1, w_ref[i], gamma, sc.b2_c if l.relu else 0, short, l.relu, x_exp=x_exp)
            bwd = oracle.layer_backward(d, e0, -12, fwd["mask"] if l.relu else np.ones_like(fwd["mask"]),
                                        fwd["x2"] if lb.x2 is not None else None, x0, b1, w_ref[i], gamma)
            want, _, _ = oracle.update(w_ref[i], bwd["g_w"], bwd["p_gw"], st.lr_mant, st.lr_exp, stochastic=True,
                                       seed=synth.BASE_SEED, step=k, tensor_id=i)
            want = want.astype(np.int8)
            changed += int(np.count_nonzero(want != w_ref[i]))
            w_ref[i] = want
            assert np.array_equal(lb.w.cpu().numpy(), want), (k, l.name)
    assert changed > 0  # the trajectory is not vacuous: updates moved weight codes

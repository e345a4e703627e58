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
    a = TrainStep(wl, h1, scalars=Scalars(), lr_mant=3, lr_exp=-4, round_mode=eoq.EOQ_ROUND_STOCHASTIC)
    b = TrainStep(wl, h2, scalars=Scalars(), lr_mant=3, lr_exp=-4, round_mode=eoq.EOQ_ROUND_STOCHASTIC)
    a.run()
    torch.cuda.synchronize()
    assert a.status() & eoq.EOQ_DEV_TIMEOUT == 0
    # the capture first runs one eager warm-up step: put weights, tables and step counter back before replaying
    w0 = [lb.w.clone() for lb in b.layers]
    b.capture(overlap=True)
    for lb, w in zip(b.layers, w0):
        lb.w.copy_(w)
    b.step_dev.zero_()
    b.weight_prep()
    for rep in range(2):  # two replays against two eager steps: scalars and step counter are read on the device
        if rep:
            a.run()
        b.replay()
        torch.cuda.synchronize()
        assert b.status() & eoq.EOQ_DEV_TIMEOUT == 0
        for la, lb in zip(a.layers, b.layers):
            for key in ("x5", "e3", "e3_exp", "g", "g_exp", "w"):
                assert torch.equal(getattr(la, key), getattr(lb, key)), (rep, la.layer.name, key)
            if la.e4 is not None:
                assert torch.equal(la.e4, lb.e4) and torch.equal(la.e4_exp, lb.e4_exp), la.layer.name
    assert b.step_dev.item() == 2
    assert any(not torch.equal(la.w, w) for la, w in zip(a.layers, w0))  # the update moved weights


def test_first_layer_of_a_step_matches_the_oracle():
    wl = workloads.get("resnet20", 2)
    st = TrainStep(wl, eoq.eoq_create(0), scalars=Scalars(), round_mode=eoq.EOQ_ROUND_STOCHASTIC)
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
        out.append((x0, e0, sc, oracle_weights(l, wl, seed, i)))
    return out


def oracle_weights(l, wl, seed, i):
    """Q_w of the Fixup-scaled Kaiming weights of layer i, formed by the oracle's own generator from the seeded
    standard-normal draws (padding input channels carry zero weights)."""
    z = synth.normal_f64((l.c_out, l.k, l.k, l.c_in), seed, 100 + i)
    wf = oracle.fixup_weights_f32(z, l.c_in_true * l.k * l.k, wl.L, wl.m, l.in_branch)
    wf[..., l.c_in_true:] = 0.0
    return oracle.q_w(wf)


@pytest.mark.parametrize("name,batch,mode", [("resnet20", 2, "rne"), ("resnet110", 1, "stochastic"), ("resnet18", 1, "stochastic"),
                                             ("resnet34", 1, "rne"), ("resnet50", 1, "stochastic")])
def test_every_layer_of_a_step_matches_the_oracle(name, batch, mode):
    """One whole step of each network at a small batch: every layer's activation, error, weight gradient
    (codes and exponents), reduction sums and updated weights against the oracle, which is fed the same seeded
    inputs generated on the host."""
    wl = workloads.get(name, batch)
    stochastic = mode == "stochastic"
    st = TrainStep(wl, eoq.eoq_create(0), scalars=Scalars(), lr_mant=3, lr_exp=-4,
                   round_mode=eoq.EOQ_ROUND_STOCHASTIC if stochastic else eoq.EOQ_ROUND_RNE)
    host = _host_inputs(st, wl)
    for lb, (_, _, _, wq) in zip(st.layers, host):
        assert np.array_equal(lb.w.cpu().numpy(), wq), lb.layer.name   # Q_w at initialisation
    st.run()
    torch.cuda.synchronize()
    assert st.status() & eoq.EOQ_DEV_TIMEOUT == 0
    sc = st.sc
    moved = 0
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
        want, _, _ = oracle.update(wq, bwd["g_w"], bwd["p_gw"], st.lr_mant, st.lr_exp, stochastic=stochastic,
                                   seed=synth.BASE_SEED, step=0, tensor_id=i)
        assert np.array_equal(lb.w.cpu().numpy().astype(np.int32), want), (l.name, "w")
        moved += int(np.count_nonzero(want != wq))
    assert moved > 0  # the update is not vacuous under either rounding


@pytest.mark.parametrize("batch,mode,replay", [(1, "stochastic", True), (2, "rne", True), (4, "stochastic", False), (2, "rne", False)])
def test_weight_trajectory_over_consecutive_steps(batch, mode, replay):
    """Small-batch online training: several consecutive steps, each with a fresh image and its own rounding draws,
    must leave after every step exactly the int8 weights the oracle reaches when it repeats the same steps.  With
    replay=True every step is a replay of one captured CUDA graph (scalars and step counter are device-resident)."""
    steps = 5
    stochastic = mode == "stochastic"
    wl = workloads.get("resnet20", batch)
    st = TrainStep(wl, eoq.eoq_create(0), scalars=Scalars(), lr_mant=3, lr_exp=-4,
                   round_mode=eoq.EOQ_ROUND_STOCHASTIC if stochastic else eoq.EOQ_ROUND_RNE)
    host = _host_inputs(st, wl)
    sc = st.sc
    w_ref = [wq.copy() for (_, _, _, wq) in host]
    if replay:
        w0 = [lb.w.clone() for lb in st.layers]
        st.capture(overlap=True)
        for lb, w in zip(st.layers, w0):
            lb.w.copy_(w)
        st.step_dev.zero_()
        st.weight_prep()
    changed = 0
    for k in range(steps):
        img = st.host_image(synth.BASE_SEED + 17 * k)   # a fresh image every step
        st.image.copy_(torch.from_numpy(img))
        if replay:
            st.replay()
        else:
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
            want, _, _ = oracle.update(w_ref[i], bwd["g_w"], bwd["p_gw"], st.lr_mant, st.lr_exp, stochastic=stochastic,
                                       seed=synth.BASE_SEED, step=k, tensor_id=i)
            want = want.astype(np.int8)
            changed += int(np.count_nonzero(want != w_ref[i]))
            w_ref[i] = want
            assert np.array_equal(lb.w.cpu().numpy(), want), (k, l.name)
    assert changed > 0  # the trajectory is not vacuous: updates moved weight codes


def test_scalars_changed_between_replays_take_effect():
    """gamma, b1 and b2 are read from device memory: a captured step follows new codes without a new capture."""
    wl = workloads.get("resnet20", 2)
    st = TrainStep(wl, eoq.eoq_create(0), scalars=Scalars())
    host = _host_inputs(st, wl)
    st.capture(overlap=True)
    new = Scalars(b1_c=4, gamma_c=97, b2_c=-6)
    st.set_scalars(new)
    w_now = [lb.w.cpu().numpy().copy() for lb in st.layers]
    st.replay()
    torch.cuda.synchronize()
    assert st.status() & eoq.EOQ_DEV_TIMEOUT == 0
    for i in (1, 3, 8):
        lb, (x0, e0, short, _) = st.layers[i], host[i]
        l = lb.layer
        d = ConvDesc(l.n, l.h, l.w, l.c_in, l.c_out, l.k, l.k, l.stride, l.pad)
        b1, gamma, b2 = st.layer_scalars(i)
        fwd = oracle.layer_forward(d, x0, b1, w_now[i], gamma, b2, short, l.relu)
        assert np.array_equal(lb.x5.cpu().numpy(), fwd["x5"]), l.name
        bwd = oracle.layer_backward(d, e0, -12, fwd["mask"] if l.relu else np.ones_like(fwd["mask"]),
                                    fwd["x2"] if lb.x2 is not None else None, x0, b1, w_now[i], gamma)
        assert np.array_equal(lb.e3.cpu().numpy(), bwd["e3"]) and lb.e3_exp.item() == bwd["p3"], l.name
        assert np.array_equal(lb.g.cpu().numpy(), bwd["g_w"]) and lb.g_exp.item() == bwd["p_gw"], l.name


FULL_SIZE_LAYERS = ["stem", "layer1.0.a", "layer2.0.a", "layer2.0.proj", "layer3.1.b"]


def test_bench_configuration_at_full_size_against_the_oracle():
    """The benchmarked workload itself (Fixup ResNet-18, batch 64, 224x224) in the launch configuration bench.py
    times (one captured graph, weight-gradient chains on side streams, replayed): a first-layer 7x7, a 3x3 of the
    first stage, a strided 3x3 with its 1x1 projection and a 256-channel 3x3 are compared with the oracle through all
    three passes and the update, element by element."""
    wl = workloads.get("resnet18", 64)
    st = TrainStep(wl, eoq.eoq_create(0), scalars=Scalars(), lr_mant=3, lr_exp=-4)
    w0 = [lb.w.clone() for lb in st.layers]
    st.capture(overlap=True)
    for lb, w in zip(st.layers, w0):
        lb.w.copy_(w)
    st.step_dev.zero_()
    st.weight_prep()
    st.replay()
    torch.cuda.synchronize()
    assert st.status() == 0
    seed, sc = synth.BASE_SEED, st.sc
    pools = {}

    def pooled(kind, shape, stream):
        if (kind, shape) not in pools:
            pools[(kind, shape)] = (synth.relu_codes if kind == "relu" else synth.normal_codes)(shape, seed, stream)
        return pools[(kind, shape)]

    for i, lb in enumerate(st.layers):
        l = lb.layer
        if l.name not in FULL_SIZE_LAYERS:
            continue
        d = ConvDesc(l.n, l.h, l.w, l.c_in, l.c_out, l.k, l.k, l.stride, l.pad)
        wq = oracle_weights(l, wl, seed, i)
        assert np.array_equal(w0[i].cpu().numpy(), wq)
        b1, gamma, b2 = st.layer_scalars(i)
        # (drawn in the order TrainStep draws them: tensors of one kind and shape share one draw)
        x_exp = -7
        if i == 0:
            img = st.host_image(seed)
            padded = np.zeros(img.shape[:3] + (l.c_in,), dtype=np.float32)
            padded[..., :img.shape[3]] = img
            codes, x_exp, _ = oracle.quantize_f32(oracle.MODE_SQ, padded)
            x0 = codes.astype(np.int8)
        else:
            x0 = pooled("relu", (l.n, l.h, l.w, l.c_in), 1)
        e0 = pooled("err", (l.n, l.ho, l.wo, l.c_out), 2)
        short = pooled("relu", (l.n, l.ho, l.wo, l.c_out), 3) if l.shortcut else None
        fwd = oracle.layer_forward(d, x0, b1, wq, gamma, b2, short, l.relu, x_exp=x_exp)
        assert np.array_equal(lb.x5.cpu().numpy(), fwd["x5"]), (l.name, "x5")
        if lb.x2 is not None:
            assert np.array_equal(lb.x2.cpu().numpy().astype(np.int32), fwd["x2"]), (l.name, "x2")
        e3, p3, s1, s2, _ = oracle.err_prescale(e0, -12, fwd["mask"] if l.relu else np.ones_like(fwd["mask"]),
                                                fwd["x2"] if lb.x2 is not None else None, gamma)
        assert np.array_equal(lb.e3.cpu().numpy(), e3) and lb.e3_exp.item() == p3, (l.name, "e3")
        assert lb.sum_e1.item() == s1
        if l.has_dgrad:
            e4, p4, _ = oracle.sq_int(oracle.conv_dgrad_acc(d, e3, wq), p3 - 7)
            assert np.array_equal(lb.e4.cpu().numpy().astype(np.int32), e4) and lb.e4_exp.item() == p4, (l.name, "e4")
            assert lb.sum_e4.item() == int(e4.astype(np.int64).sum())
        g, pg, _ = oracle.sq_int(oracle.conv_wgrad_acc(d, e3, x0, b1), p3 - 7)
        assert np.array_equal(lb.g.cpu().numpy().astype(np.int32), g) and lb.g_exp.item() == pg, (l.name, "g_w")
        want, _, _ = oracle.update(wq, g.astype(np.int8), pg, st.lr_mant, st.lr_exp, stochastic=False)
        assert np.array_equal(lb.w.cpu().numpy().astype(np.int32), want), (l.name, "w")

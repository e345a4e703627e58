"""The closed-loop training step on the GPU (every unit chained to its neighbours, pooling, error joins, float head,
scalar and weight updates) against the oracle's closed-loop step: every intermediate tensor of every unit, the
head's results and every updated parameter, bit for bit (the reported loss within 1e-6 relative: its logarithm is
each side's library routine)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import network as N
from paper_2105_13890_b200 import eoq, synth, workloads
from paper_2105_13890_b200.chain import ChainedStep
from paper_2105_13890_b200.step import Scalars

pytestmark = pytest.mark.gpu

SEED = synth.BASE_SEED


def build(name, batch, round_mode, lr=(3, -4), keep_pool_error=False):
    if name == "resnet20":
        wl, classes, pool = workloads.resnet20(batch), 10, None
        net = N.resnet20(batch)
    else:
        wl, classes, pool = workloads.resnet18(batch), 1000, (3, 2, 1)
        net = N.resnet18(batch)
    st = ChainedStep(wl, eoq.eoq_create(0), scalars=Scalars(), lr_mant=lr[0], lr_exp=lr[1], head_lr=2.0 ** -6, classes=classes,
                     pool=pool, round_mode=round_mode, seed=SEED, keep_pool_error=keep_pool_error)
    N.init(net, lambda s, stream: synth.normal_f64(s, SEED, stream), lambda s, stream: synth.normal_f32(s, SEED, stream),
           b1=-2, gamma=118, b2=3)
    return wl, st, net


def feed(st, k):
    """A fresh seeded image and labels for step k, on both sides."""
    f = st.units[0].layer
    img = synth.normal_f32((f.n, f.h, f.w, 3), SEED + 31 * k, 0)
    labels = synth.labels(f.n, st.classes, SEED + 31 * k, 1).astype(np.int32)
    st.image.copy_(torch.from_numpy(img))
    st.labels.copy_(torch.from_numpy(labels))
    return img, labels


def host(t):
    return t.cpu().numpy()


def compare_parameters(st, net, where):
    for u, ou in zip(st.units, net.units):
        assert np.array_equal(host(u.w), ou.w), (where, ou.name, "w")
        assert host(u.scal).tolist() == [ou.b1 if u.role != "proj" else net.units[u.index - 1].b1, ou.gamma, ou.b2], (where, ou.name, "scalars")
    assert np.array_equal(host(st.W), net.W) and np.array_equal(host(st.bias), net.bias), (where, "head")


@pytest.mark.parametrize("name,batch,mode", [("resnet20", 2, eoq.EOQ_ROUND_RNE), ("resnet20", 4, eoq.EOQ_ROUND_STOCHASTIC),
                                             ("resnet18", 2, eoq.EOQ_ROUND_RNE)])
def test_chained_step_matches_the_oracle_on_every_tensor(name, batch, mode):
    wl, st, net = build(name, batch, mode, keep_pool_error=True)
    compare_parameters(st, net, "init")
    img, labels = feed(st, 0)
    st.run()
    torch.cuda.synchronize()
    assert st.status() & ~eoq.EOQ_DEV_SQ_ZERO == 0
    log = N.train_step(net, img, labels, st.lr_mant, st.lr_exp, st.head_lr, stochastic=mode == eoq.EOQ_ROUND_STOCHASTIC, seed=SEED)
    hd = log["head"]
    m = st.units[0].wmargin
    f = st.units[0].layer
    assert np.array_equal(host(st.units[0].x0)[:, :, m:m + f.w, :], hd["x_in"]) and st.image_exp.item() == hd["p_in"]
    for u, ou in zip(st.units, net.units):
        fw, bw = log[ou.name]["fwd"], log[ou.name]["bwd"]
        assert np.array_equal(host(u.x5), fw["x5"]), (ou.name, "x5")
        if u.x2 is not None:
            assert np.array_equal(host(u.x2).astype(np.int32), fw["x2"]), (ou.name, "x2")
        assert np.array_equal(host(u.e3), bw["e3"]) and u.e3_exp.item() == bw["p3"], (ou.name, "e3")
        assert u.sum_e1.item() == bw["sum_e1"], (ou.name, "sum_e1")
        if u.role != "stem":
            assert np.array_equal(host(u.e4), bw["e4"]) and u.e4_exp.item() == bw["p4"], (ou.name, "e4")
            assert u.sum_e4.item() == bw["sum_e4"], (ou.name, "sum_e4")
        if u.role == "b":
            assert u.sum_e1x2.item() == bw["sum_e1x2"], (ou.name, "sum_e1x2")
        assert np.array_equal(host(u.g), bw["g_w"]) and u.g_exp.item() == bw["p_gw"], (ou.name, "g_w")
    for blk, ob in zip(st.blocks, net.blocks):
        bw = log[net.units[ob.a].name]["bwd"]
        assert np.array_equal(host(blk.e_in), bw["join"]) and blk.e_in_exp.item() == bw["p_join"], (blk.a.layer.name, "join")
        assert blk.sum_join.item() == bw["sum_join"]
    if st.pool:
        assert np.array_equal(host(st.stem_e0), log["pool"]["e"]) and st.stem_e0_exp.item() == log["pool"]["p"]
    assert np.array_equal(host(st.sums).astype(np.int64), hd["sums"])
    assert np.array_equal(host(st.logits), hd["logits"])                 # fp32, bit for bit
    assert np.array_equal(host(st.dpooled), hd["dpooled"])
    assert st.loss.item() == pytest.approx(hd["loss"], rel=1e-6)
    assert np.array_equal(host(st.e_head), hd["e"]) and st.e_head_exp.item() == hd["p_e"]
    which = {"b1": 0, "gamma": 1, "b2": 2}
    for (uname, w), (code, p) in log["scalar_grads"].items():
        u = next(x for x, ou in zip(st.units, net.units) if ou.name == uname)
        assert host(u.sgrad[which[w]]).tolist() == [code, p], (uname, w)
    compare_parameters(st, net, "after the step")


def test_closed_loop_step_at_the_benchmark_size():
    """Fixup ResNet-18 at batch 64, 224x224, in the configuration the benchmark times (one captured graph with the
    weight-gradient work on side streams, replayed): every unit's error codes and weight gradient, the joined errors,
    the head's results and every updated parameter against the oracle (which needs about a minute for this step)."""
    wl, st, net = build("resnet18", 64, eoq.EOQ_ROUND_RNE, lr=(1, -8))
    saved = st.save()
    feed(st, 0)
    st.capture(overlap=True)
    st.restore(saved)
    img, labels = feed(st, 1)
    st.replay()
    torch.cuda.synchronize()
    assert st.status() & ~eoq.EOQ_DEV_SQ_ZERO == 0
    log = N.train_step(net, img, labels, st.lr_mant, st.lr_exp, st.head_lr, stochastic=False, seed=SEED)
    for u, ou in zip(st.units, net.units):
        fw, bw = log[ou.name]["fwd"], log[ou.name]["bwd"]
        assert np.array_equal(host(u.x5), fw["x5"]), (ou.name, "x5")
        assert np.array_equal(host(u.e3), bw["e3"]) and u.e3_exp.item() == bw["p3"], (ou.name, "e3")
        assert np.array_equal(host(u.g), bw["g_w"]) and u.g_exp.item() == bw["p_gw"], (ou.name, "g_w")
    for blk, ob in zip(st.blocks, net.blocks):
        bw = log[net.units[ob.a].name]["bwd"]
        assert np.array_equal(host(blk.e_in), bw["join"]) and blk.e_in_exp.item() == bw["p_join"], (blk.a.layer.name, "join")
    assert np.array_equal(host(st.logits), log["head"]["logits"]) and np.array_equal(host(st.dpooled), log["head"]["dpooled"])
    compare_parameters(st, net, "after the step")


def run_trajectory(name, batch, steps, mode, full_at):
    """`steps` consecutive closed-loop steps replayed from one captured graph, a fresh image and labels every step:
    checksum of the parameters every step, full tensors at the steps in `full_at`."""
    wl, st, net = build(name, batch, mode, lr=(1, -8))   # a rate at which the scalars stay in range at 224x224
    saved = st.save()
    feed(st, 0)
    st.capture(overlap=True)      # runs one real step as warm-up: put the parameters back
    st.restore(saved)
    assert st.status() & ~eoq.EOQ_DEV_SQ_ZERO == 0
    start = [u.w.copy() for u in net.units]
    for k in range(steps):
        img, labels = feed(st, k)
        st.replay()
        torch.cuda.synchronize()
        assert st.status() & ~eoq.EOQ_DEV_SQ_ZERO == 0
        N.train_step(net, img, labels, st.lr_mant, st.lr_exp, st.head_lr, stochastic=mode == eoq.EOQ_ROUND_STOCHASTIC, seed=SEED,
                     keep=False)
        for u, ou in zip(st.units, net.units):   # the int8 weight trajectory, every step
            assert np.array_equal(host(u.w), ou.w), (k, ou.name)
        if k + 1 in full_at:
            compare_parameters(st, net, f"step {k + 1}")
    changed = sum(int(np.count_nonzero(ou.w != w0)) for ou, w0 in zip(net.units, start))
    total = sum(ou.w.size for ou in net.units)
    return changed / total


@pytest.mark.parametrize("batch,steps", [(1, 10), (2, 10), (4, 5)])
def test_small_batch_online_training_first_steps(batch, steps):
    """Fixup ResNet-18 at batch 1, 2 and 4 (224x224 synthetic images): consecutive int8 training steps as graph
    replays, the weight trajectory bit-exact after every step (the oracle needs seconds per step; the full 100
    steps run under -m 'gpu and slow')."""
    frac = run_trajectory("resnet18", batch, steps, eoq.EOQ_ROUND_STOCHASTIC, full_at=(1, steps))
    assert frac > 1e-3     # the run is not vacuous: more than one weight code in a thousand moved


@pytest.mark.slow
@pytest.mark.parametrize("batch", [1, 2, 4])
def test_small_batch_online_training_hundred_steps(batch):
    """The full length of the small-batch configuration: 100 steps (minutes of oracle time; run with -m 'gpu and slow')."""
    frac = run_trajectory("resnet18", batch, 100, eoq.EOQ_ROUND_STOCHASTIC, full_at=(1, 10, 100))
    assert frac > 1e-2

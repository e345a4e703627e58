"""A whole Fixup ResNet training step on the oracle (test infrastructure, not product code).

Strings the layer units of ``eoq_oracle`` together the way Sec. 3.2.1 of arXiv 2105.13890 chains them
(x0 of a layer is x5 of the one before, e0 of a layer is the error its successor hands back), with the glue the
paper leaves open written out as conventions of this build:

  * a basic block is unit A (bias b1, 3x3 conv, gamma fixed at 1, bias b2, ReLU) followed by unit B (b1, 3x3 conv,
    trainable gamma, b2, + shortcut, ReLU); the shortcut joins at x4 of unit B.  A stage entry with a stride or a
    channel change has a 1x1 projection unit P (gamma 1, no b2, no ReLU) fed by the same x0 + b1 as unit A;
  * the error leaving unit B through the shortcut is e1 of unit B (the error at x4); where it meets the error of
    the branch (block input), the two are added exactly at the smaller exponent and requantized with Q_e; a bias
    whose x1 feeds both a branch and a projection takes g_b1 from the joined error, otherwise from e4 of its unit;
  * the first layer takes SQ(image), has no b1 and no error output; the ImageNet networks max-pool after it;
  * global average pooling, a float linear layer and softmax cross-entropy close the network (Sec. 5.1 keeps the
    last layer unquantized); the error of the pooled activations, divided by the number of positions, is
    quantized with Q_e and spread over the positions;
  * every parameter is updated by the rule of Sec. 3.2.3: weights saturate at +-127 (Q_w = CQ), gamma and the
    biases at the 16-bit range (Q), the linear layer takes a plain fp32 SGD step.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

from . import eoq_oracle as O
from .eoq_oracle import ConvDesc


@dataclass
class Unit:
    name: str
    d: ConvDesc
    c_in_true: int
    role: str                    # "stem", "a", "b", "proj"
    relu: bool = True
    in_branch: bool = True
    # parameters (integer codes at p = -7)
    w: Optional[np.ndarray] = None
    b1: int = 0
    gamma: int = 128
    b2: int = 0


@dataclass
class Block:
    a: int                       # index of unit A
    b: int                       # index of unit B
    proj: Optional[int] = None   # index of the projection unit


@dataclass
class Net:
    units: List[Unit]
    blocks: List[Block]
    pool: Optional[tuple]        # (k, s, p) of the max-pool behind the first layer, or None
    classes: int
    L: int
    m: int
    W: Optional[np.ndarray] = None      # fp32 [classes, c]
    bias: Optional[np.ndarray] = None
    step_no: int = 0
    log: Dict[str, dict] = field(default_factory=dict)


def _out(h, k, s, p):
    return (h + 2 * p - k) // s + 1


def resnet_basic(batch: int, image: int, stem: tuple, stem_c: int, pool, widths, blocks, classes: int) -> Net:
    """Fixup ResNet of basic blocks.  stem = (k, stride, pad); stem_c = stored input channels (3 real)."""
    units: List[Unit] = []
    blks: List[Block] = []
    k, s, p = stem
    units.append(Unit("stem", ConvDesc(batch, image, image, stem_c, widths[0], k, k, s, p), 3, "stem", in_branch=False))
    h = _out(image, k, s, p)
    if pool:
        h = _out(h, *pool)
    c = widths[0]
    for si, (co, nb) in enumerate(zip(widths, blocks)):
        for bi in range(nb):
            st = (1 if si == 0 else 2) if bi == 0 else 1
            ci = c if bi == 0 else co
            ia = len(units)
            units.append(Unit(f"s{si}.{bi}.a", ConvDesc(batch, h, h, ci, co, 3, 3, st, 1), ci, "a"))
            ip = None
            if st != 1 or ci != co:
                ip = len(units)
                units.append(Unit(f"s{si}.{bi}.proj", ConvDesc(batch, h, h, ci, co, 1, 1, st, 0), ci, "proj", relu=False, in_branch=False))
            h = _out(h, 3, st, 1)
            ib = len(units)
            units.append(Unit(f"s{si}.{bi}.b", ConvDesc(batch, h, h, co, co, 3, 3, 1, 1), co, "b"))
            blks.append(Block(ia, ib, ip))
        c = co
    return Net(units, blks, pool, classes, L=sum(blocks), m=2)


def resnet18(batch: int, image: int = 224, classes: int = 1000, stem_c: int = 8) -> Net:
    return resnet_basic(batch, image, (7, 2, 3), stem_c, (3, 2, 1), (64, 128, 256, 512), (2, 2, 2, 2), classes)


def resnet34(batch: int, image: int = 224, classes: int = 1000, stem_c: int = 8) -> Net:
    return resnet_basic(batch, image, (7, 2, 3), stem_c, (3, 2, 1), (64, 128, 256, 512), (3, 4, 6, 3), classes)


def resnet20(batch: int, image: int = 32, classes: int = 10, stem_c: int = 16) -> Net:
    return resnet_basic(batch, image, (3, 1, 1), stem_c, None, (16, 32, 64), (3, 3, 3), classes)


def resnet110(batch: int, image: int = 32, classes: int = 10, stem_c: int = 16) -> Net:
    return resnet_basic(batch, image, (3, 1, 1), stem_c, None, (16, 32, 64), (18, 18, 18), classes)


def init(net: Net, normal_f64, normal_f32, b1: int = 0, gamma: int = 128, b2: int = 0) -> None:
    """Fixup-scaled Kaiming weights through Q_w, scalars at the given codes, N(0, 1/c) linear layer.
    normal_f64(shape, stream) / normal_f32(shape, stream) supply the seeded standard-normal draws."""
    for i, u in enumerate(net.units):
        d = u.d
        z = normal_f64((d.c_out, d.kh, d.kw, d.c_in), 100 + i)
        wf = O.fixup_weights_f32(z, u.c_in_true * d.kh * d.kw, net.L, net.m, u.in_branch)
        wf[..., u.c_in_true:] = 0.0
        u.w = O.q_w(wf)
        u.b1 = 0 if u.role == "stem" else b1
        u.gamma = gamma if u.role == "b" else 128
        u.b2 = 0 if u.role == "proj" else b2
    c = net.units[-1].d.c_out
    net.W = (normal_f32((net.classes, c), 500) * np.float32(1.0 / np.sqrt(c))).astype(np.float32)
    net.bias = np.zeros(net.classes, dtype=np.float32)


def _scalar_update(theta: int, total: int, p_total: int, lr, mode, tid: int, step: int) -> tuple:
    """One scalar parameter: g = Q_g({total}), theta <- Q(theta - Q_u(lr g)) on the 16-bit range."""
    g, pg, zero = O.sq_int(np.array([total], dtype=np.int64), p_total)
    lr_mant, lr_exp, seed = lr
    new, _, _ = O.update(np.array([theta], dtype=np.int32), g.astype(np.int8), pg, lr_mant, lr_exp, lo=-32768, hi=32767,
                         stochastic=mode, seed=seed, step=step, tensor_id=tid)
    return int(new[0]), (int(g[0]), pg)


def forward_trunk(net: Net, x_in: np.ndarray, p_in: int):
    """Forward chain of every unit.  -> (per-unit forward results, per-unit x0, last activation, max-pool indices)."""
    units = net.units
    stem = units[0]
    fw: Dict[int, dict] = {}
    x0s: Dict[int, np.ndarray] = {0: x_in}
    f = O.layer_forward(stem.d, x_in, 0, stem.w, stem.gamma, stem.b2, None, True, x_exp=p_in)
    fw[0] = f
    x = f["x5"]
    pool_idx = None
    if net.pool:
        x, pool_idx = O.maxpool_fwd(x, *net.pool)
    for blk in net.blocks:
        ua, ub = units[blk.a], units[blk.b]
        x0s[blk.a] = x
        fa = O.layer_forward(ua.d, x, ua.b1, ua.w, ua.gamma, ua.b2, None, True)
        fw[blk.a] = fa
        if blk.proj is not None:
            up = units[blk.proj]
            x0s[blk.proj] = x
            fp = O.layer_forward(up.d, x, ua.b1, up.w, 128, 0, None, False)   # fed by unit A's x0 + b1
            fw[blk.proj] = fp
            short = fp["x5"]
        else:
            short = x
        x0s[blk.b] = fa["x5"]
        fb = O.layer_forward(ub.d, fa["x5"], ub.b1, ub.w, ub.gamma, ub.b2, short, True)
        fw[blk.b] = fb
        x = fb["x5"]
    return fw, x0s, x, pool_idx


def backward_trunk(net: Net, fw, x0s, pool_idx, e_out: np.ndarray, p_out: int):
    """Error chain from the error of the last activation back to the first layer.
    -> (per-unit backward results, [(unit, g_w, exponent)], [(unit, scalar name, exact sum, exponent)], pool log)."""
    units = net.units
    stem = units[0]
    grads, scal = [], []
    bw: Dict[int, dict] = {}
    for blk in reversed(net.blocks):
        ua, ub = units[blk.a], units[blk.b]
        fb, fa = fw[blk.b], fw[blk.a]
        bb = O.layer_backward(ub.d, e_out, p_out, fb["mask"], fb["x2"], x0s[blk.b], ub.b1, ub.w, ub.gamma)
        bw[blk.b] = bb
        grads.append((blk.b, bb["g_w"], bb["p_gw"]))
        scal += [(blk.b, "b1", bb["sum_e4"], bb["p4"]), (blk.b, "b2", bb["sum_e1"], p_out), (blk.b, "gamma", bb["sum_e1x2"], p_out - 7)]
        ba = O.layer_backward(ua.d, bb["e4"], bb["p4"], fa["mask"], None, x0s[blk.a], ua.b1, ua.w, 128)
        bw[blk.a] = ba
        grads.append((blk.a, ba["g_w"], ba["p_gw"]))
        scal.append((blk.a, "b2", ba["sum_e1"], bb["p4"]))
        if blk.proj is not None:
            up = units[blk.proj]
            # the error entering the shortcut is e1 of unit B: e_out gated by unit B's ReLU mask
            bp = O.layer_backward(up.d, e_out, p_out, fb["mask"], None, x0s[blk.proj], ua.b1, up.w, 128)
            bw[blk.proj] = bp
            grads.append((blk.proj, bp["g_w"], bp["p_gw"]))
            S, pj = O.join(ba["e4"], ba["p4"], bp["e4"], bp["p4"])
        else:
            S, pj = O.join(ba["e4"], ba["p4"], e_out, p_out, fb["mask"])
        ej, p_j, _ = O.sq_int(S, pj)
        ba["join_acc"], ba["join_acc_exp"] = S, pj
        ba["join"], ba["p_join"] = ej.astype(np.int8), p_j
        ba["sum_join"] = int(ej.astype(np.int64).sum())
        if blk.proj is not None:
            scal.append((blk.a, "b1", ba["sum_join"], p_j))
        else:
            scal.append((blk.a, "b1", ba["sum_e4"], ba["p4"]))
        e_out, p_out = ej.astype(np.int8), p_j
    pool_log = None
    if net.pool:
        S = O.maxpool_bwd(e_out, pool_idx, fw[0]["x5"].shape)
        ep, p_out, _ = O.sq_int(S, p_out)
        e_out = ep.astype(np.int8)
        pool_log = {"e": e_out, "p": p_out}
    e3, p3, s1, _, _ = O.err_prescale(e_out, p_out, fw[0]["mask"], None, 128)
    G = O.conv_wgrad_acc(stem.d, e3, x0s[0], 0)
    g, pg, _ = O.sq_int(G, p3 - 7)
    bw[0] = {"e0": e_out, "p0": p_out, "e3": e3, "p3": p3, "g_w": g.astype(np.int8), "p_gw": pg, "sum_e1": s1}
    grads.append((0, g.astype(np.int8), pg))
    scal.append((0, "b2", s1, p_out))
    return bw, grads, scal, pool_log


def train_step(net: Net, image_f32: np.ndarray, labels: np.ndarray, lr_mant: int, lr_exp: int, head_lr: float,
               stochastic: bool = False, seed: int = 0, keep: bool = True) -> dict:
    """One closed-loop training step; parameters are updated in place.  Returns every intermediate tensor by unit
    name (when keep is set) plus the head's results."""
    units, log = net.units, {}
    stem = units[0]
    n = stem.d.n
    padded = np.zeros((n, stem.d.h, stem.d.w, stem.d.c_in), dtype=np.float32)
    padded[..., :image_f32.shape[3]] = image_f32
    codes, p_in, _ = O.quantize_f32(O.MODE_SQ, padded)
    x_in = codes.astype(np.int8)

    fw, x0s, x, pool_idx = forward_trunk(net, x_in, p_in)
    hw = x.shape[1] * x.shape[2]
    sums = O.avgpool_sum(x)
    loss, dpooled, logits = O.head(sums, hw, net.W, net.bias, labels, head_lr)
    e_f = (dpooled / np.float32(hw)).astype(np.float32)
    ec, p_e, _ = O.quantize_f32(O.MODE_SQ, e_f)
    e_out = np.broadcast_to(ec.astype(np.int8)[:, None, None, :], x.shape).copy()
    log["head"] = {"sums": sums, "logits": logits, "loss": loss, "dpooled": dpooled, "e": e_out, "p_e": p_e, "p_in": p_in,
                   "x_in": x_in}

    bw, grads, scal, pool_log = backward_trunk(net, fw, x0s, pool_idx, e_out, p_e)
    if pool_log:
        log["pool"] = pool_log

    # ---------------- update (Sec. 3.2.3)
    lr = (lr_mant, lr_exp, seed)
    for i, g, pg in grads:
        new, _, _ = O.update(units[i].w, g, pg, lr_mant, lr_exp, stochastic=stochastic, seed=seed, step=net.step_no, tensor_id=i)
        units[i].w = new.astype(np.int8)
    which_id = {"b1": 0, "gamma": 1, "b2": 2}
    sgrads = {}
    for i, which, total, p_tot in scal:
        u = units[i]
        new, gq = _scalar_update(getattr(u, which), total, p_tot, lr, stochastic, 1000 + 3 * i + which_id[which], net.step_no)
        setattr(u, which, new)
        sgrads[(u.name, which)] = gq
    net.step_no += 1
    if keep:
        for i, u in enumerate(units):
            log[u.name] = {"fwd": fw[i], "bwd": bw[i], "x0": x0s[i]}
    log["scalar_grads"] = sgrads
    return log

"""A closed-loop training step of a Fixup ResNet of basic blocks through the C ABI (buffer plumbing only).

Every quantized convolution unit runs the library's forward / error-head / dgrad / wgrad calls exactly as in
``step.py``, but here the units are chained as Sec. 3.2.1 of arXiv 2105.13890 chains them: the input of a unit is
the activation its predecessor wrote, its incoming error is what its successor propagated back.  The glue between
units goes through the ``eoq_aux_*`` entry points: max-pooling behind an ImageNet first layer, global average
pooling, the floating-point last layer with softmax cross-entropy, the quantized error it hands back, the exact
join of branch and shortcut errors at a block input, and the update of gamma and the biases next to the 8-bit
weight update.  Scalars, step counter, image and labels live in device memory, so one captured CUDA graph performs
consecutive training steps.

Block structure (read off the workload's layer names ``<stage>.<block>.a | .proj | .b``): unit A (b1, 3x3 conv, b2,
ReLU), optional 1x1 projection fed by the same x0 + b1, unit B (b1, 3x3 conv, gamma, b2, + shortcut at x4, ReLU).
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from . import eoq, synth
from .step import Scalars
from .workloads import Layer, Workload, init_weight_f32


class UnitBuffers:
    def __init__(self, index: int, layer: Layer, dev, wmargin: int = 0):
        self.index, self.layer, self.wmargin = index, layer, wmargin
        l = layer
        self.desc = eoq.conv_desc(l.n, l.h, l.w, l.c_in, l.c_out, l.k, l.k, l.stride, l.pad, wmargin)
        i8 = torch.int8
        out = (l.n, l.ho, l.wo, l.c_out)
        self.role = "stem" if index == 0 else l.name.rsplit(".", 1)[1]
        self.w = torch.empty((l.c_out, l.k, l.k, l.c_in), dtype=i8, device=dev)
        self.x5 = torch.empty(out, dtype=i8, device=dev)
        self.n_out = int(np.prod(out))
        self.x2 = torch.empty(out, dtype=torch.int16, device=dev) if self.role == "b" else None
        self.mask = torch.empty((self.n_out + 7) // 8, dtype=torch.uint8, device=dev) if l.relu else None
        self.e3 = torch.empty(out, dtype=i8, device=dev)
        self.e3_exp = torch.zeros(1, dtype=torch.int32, device=dev)
        self.e4 = torch.empty((l.n, l.h, l.w, l.c_in), dtype=i8, device=dev) if l.has_dgrad else None
        self.e4_exp = torch.zeros(1, dtype=torch.int32, device=dev)
        self.sum_e4 = torch.zeros(1, dtype=torch.int64, device=dev)
        self.sum_e1 = torch.zeros(1, dtype=torch.int64, device=dev)
        self.sum_e1x2 = torch.zeros(1, dtype=torch.int64, device=dev)
        self.g = torch.empty_like(self.w)
        self.g_exp = torch.zeros(1, dtype=torch.int32, device=dev)
        self.scal = torch.zeros(3, dtype=torch.int32, device=dev)      # {b1, gamma, b2}
        self.sgrad = torch.zeros((3, 2), dtype=torch.int32, device=dev)  # Q_g of the three scalar gradients: {code, exponent}
        self.prep = torch.empty(max(eoq.eoq_weight_prep_size(self.desc), 256), dtype=torch.uint8, device=dev)
        self.x0 = None          # set when the units are chained
        self.e0 = None          # (codes, exponent tensor) of the incoming error
        self.e0_exp = None


class BlockBuffers:
    def __init__(self, a: UnitBuffers, b: UnitBuffers, proj: Optional[UnitBuffers], dev):
        self.a, self.b, self.proj = a, b, proj
        l = a.layer
        self.e_in = torch.empty((l.n, l.h, l.w, l.c_in), dtype=torch.int8, device=dev)   # joined error at the block input
        self.e_in_exp = torch.zeros(1, dtype=torch.int32, device=dev)
        self.sum_join = torch.zeros(1, dtype=torch.int64, device=dev)


class ChainedStep:
    """Device buffers of a whole network at one batch size and the calls of one closed-loop training step."""

    def __init__(self, workload: Workload, handle: int, device: str = "cuda:0", seed: int = synth.BASE_SEED,
                 scalars: Optional[Scalars] = None, lr_mant: int = 3, lr_exp: int = -4, head_lr: float = 2.0 ** -6,
                 classes: int = 1000, pool: Optional[tuple] = None, round_mode: int = eoq.EOQ_ROUND_RNE,
                 image_channels: int = 3, side_streams: int = 2, keep_pool_error: bool = False, finish_together: bool = True):
        self.wl, self.h, self.dev = workload, handle, torch.device(device)
        self.keep_pool_error = keep_pool_error   # also write the error between the pool and the first layer's head
        # weight gradients: only the GEMMs run per layer beside the backward chain; the b1 sums, slice sums and Q_g of all
        # layers follow in four launches at the end (each layer then keeps its sums in a workspace of its own)
        self.finish_together = finish_together
        self.sc = scalars or Scalars()
        self.lr_mant, self.lr_exp, self.head_lr, self.classes = lr_mant, lr_exp, head_lr, classes
        self.round_mode, self.seed, self.pool = round_mode, seed, pool
        dev = self.dev
        layers = workload.layers
        first_margin = 5 if layers[0].k >= 5 else 0
        self.units: List[UnitBuffers] = [UnitBuffers(i, l, dev, first_margin if i == 0 else 0) for i, l in enumerate(layers)]
        # blocks from the layer names
        self.blocks: List[BlockBuffers] = []
        i = 1
        while i < len(self.units):
            a = self.units[i]
            assert a.role == "a", a.layer.name
            proj = self.units[i + 1] if self.units[i + 1].role == "proj" else None
            b = self.units[i + (2 if proj else 1)]
            assert b.role == "b"
            self.blocks.append(BlockBuffers(a, b, proj, dev))
            i += 3 if proj else 2
        stem = self.units[0]
        fl = stem.layer
        self.image_channels = image_channels
        self.image = torch.zeros((fl.n, fl.h, fl.w, image_channels), dtype=torch.float32, device=dev)
        self.image_exp = torch.zeros(1, dtype=torch.int32, device=dev)
        stem.x0 = torch.zeros((fl.n, fl.h, fl.w + 2 * first_margin, fl.c_in), dtype=torch.int8, device=dev)
        self.labels = torch.zeros(fl.n, dtype=torch.int32, device=dev)
        # max-pool behind the first layer
        x = stem.x5
        if pool:
            k, s, p = pool
            hp = (fl.ho + 2 * p - k) // s + 1
            self.pooled = torch.empty((fl.n, hp, hp, fl.c_out), dtype=torch.int8, device=dev)
            self.pool_arg = torch.empty((fl.n, hp, hp, fl.c_out), dtype=torch.uint8, device=dev)
            x = self.pooled
        # chain the activations
        for blk in self.blocks:
            blk.a.x0 = x
            if blk.proj:
                blk.proj.x0 = x
            blk.b.x0 = blk.a.x5
            blk.shortcut = blk.proj.x5 if blk.proj else x
            blk.b.shortcut = blk.shortcut
            x = blk.b.x5
        last = self.blocks[-1].b.layer
        self.hw, self.c_last = last.ho * last.wo, last.c_out
        n = fl.n
        self.sums = torch.zeros((n, self.c_last), dtype=torch.int32, device=dev)
        self.W = torch.empty((classes, self.c_last), dtype=torch.float32, device=dev)
        self.bias = torch.zeros(classes, dtype=torch.float32, device=dev)
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
        self.dpooled = torch.zeros((n, self.c_last), dtype=torch.float32, device=dev)
        self.logits = torch.zeros((n, classes), dtype=torch.float32, device=dev)
        self.head_ws = torch.empty(eoq.eoq_aux_head_workspace_size(n, self.c_last, classes), dtype=torch.uint8, device=dev)
        self.e_head = torch.empty((n, last.ho, last.wo, self.c_last), dtype=torch.int8, device=dev)
        self.e_head_exp = torch.zeros(1, dtype=torch.int32, device=dev)
        self.stem_e0 = torch.empty((fl.n, fl.ho, fl.wo, fl.c_out), dtype=torch.int8, device=dev) if pool else None
        self.stem_e0_exp = torch.zeros(1, dtype=torch.int32, device=dev)
        self.c128 = torch.tensor([128], dtype=torch.int32, device=dev)   # gamma of a projection's error head
        self.step_dev = torch.zeros(1, dtype=torch.int64, device=dev)
        # workspaces: conv passes, pooling backward (int32 sums), head error (floats)
        ws = 256
        for u in self.units:
            for p_ in (eoq.EOQ_PASS_DGRAD, eoq.EOQ_PASS_WGRAD):
                ws = max(ws, eoq.eoq_workspace_size(u.desc, p_))
        ws = max(ws, n * self.c_last * 4)
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=dev)
        dev_index = dev.index if dev.index is not None else 0
        self.h_sides = [eoq.eoq_create(dev_index) for _ in range(side_streams)]
        self.workspace_sides = [torch.empty(ws, dtype=torch.uint8, device=dev) for _ in range(side_streams)]
        half = torch.cuda.get_device_properties(dev).multi_processor_count // 2
        for hs in self.h_sides:
            eoq.eoq_set_gemm_ctas(hs, half)
        self.sides = [torch.cuda.Stream(device=dev) for _ in range(side_streams)]
        if finish_together:
            for u in self.units:
                u.wgrad_ws = torch.empty(max(256, eoq.eoq_workspace_size(u.desc, eoq.EOQ_PASS_WGRAD)), dtype=torch.uint8, device=dev)
                u.wgrad_parts = 0
                u.b1_dev = None
        self.graph = None
        self._init_parameters(seed)
        self._scalar_items()

    # ------------------------------------------------------------------ parameters
    def _init_parameters(self, seed: int) -> None:
        sc = self.sc
        for u in self.units:
            l = u.layer
            wf = init_weight_f32(l, self.wl, synth.normal_f64(tuple(u.w.shape), seed, 100 + u.index))
            wf_d = torch.from_numpy(wf).to(self.dev)
            eoq.eoq_quantize(self.h, eoq.EOQ_CQ, wf_d, True, None, wf_d.numel(), u.w)   # Q_w, once at initialisation
            b1 = 0 if u.role == "stem" else sc.b1_c
            gamma = sc.gamma_c if u.role == "b" else 128
            b2 = 0 if u.role == "proj" else sc.b2_c
            u.scal.copy_(torch.tensor([b1, gamma, b2], dtype=torch.int32))
        Wf = (synth.normal_f32((self.classes, self.c_last), seed, 500) * np.float32(1.0 / np.sqrt(self.c_last))).astype(np.float32)
        self.W.copy_(torch.from_numpy(Wf))
        self.bias.zero_()
        self.weight_prep()
        torch.cuda.synchronize(self.dev)

    def weight_prep(self) -> None:
        eoq.eoq_weight_prep(self.h, [u.desc for u in self.units], [u.w for u in self.units], [u.prep for u in self.units])

    def _scalar_items(self) -> None:
        """The trainable scalars with the sums and exponents their gradients are formed from (ids: 1000 + 3 unit + k,
        k = 0 for b1, 1 for gamma, 2 for b2)."""
        items = []   # (theta, mirror, total, exponent tensor, exponent bias, tensor id, grad out)

        def add(u, k, total, exp, bias, mirror=None):
            items.append((u.scal[k:k + 1], mirror, total, exp, bias, 1000 + 3 * u.index + k, u.sgrad[k]))

        nxt_e, nxt_exp = self.e_head, self.e_head_exp
        for blk in reversed(self.blocks):
            a, b, pr = blk.a, blk.b, blk.proj
            add(b, 0, b.sum_e4, b.e4_exp, 0)
            add(b, 2, b.sum_e1, nxt_exp, 0)
            add(b, 1, b.sum_e1x2, nxt_exp, -7)
            add(a, 2, a.sum_e1, b.e4_exp, 0)
            if pr:
                add(a, 0, blk.sum_join, blk.e_in_exp, 0, mirror=pr.scal[0:1])   # the projection reads unit A's b1
            else:
                add(a, 0, a.sum_e4, a.e4_exp, 0)
            nxt_e, nxt_exp = blk.e_in, blk.e_in_exp
        stem = self.units[0]
        add(stem, 2, stem.sum_e1, self.stem_e0_exp if self.pool else nxt_exp, 0)
        self.items = items

    # ------------------------------------------------------------------ one step
    def run(self, overlap: bool = False) -> None:
        h, ws = self.h, self.workspace
        main = torch.cuda.current_stream(self.dev)
        stem = self.units[0]
        fl = stem.layer
        eoq.eoq_quantize_image(h, self.image, fl.n, fl.h, fl.w, self.image_channels, fl.c_in, stem.wmargin, stem.x0, self.image_exp)
        eoq.eoq_conv_fwd_dev(h, stem.desc, stem.x0, self.image_exp, stem.scal, stem.w, stem.prep, None, True, stem.x5, None, stem.mask)
        if self.pool:
            k, s, p = self.pool
            eoq.eoq_aux_maxpool_fwd(h, stem.x5, fl.n, fl.ho, fl.wo, fl.c_out, k, s, p, self.pooled, self.pool_arg)
        for blk in self.blocks:
            a, b, pr = blk.a, blk.b, blk.proj
            eoq.eoq_conv_fwd_dev(h, a.desc, a.x0, None, a.scal, a.w, a.prep, None, True, a.x5, None, a.mask)
            if pr:
                eoq.eoq_conv_fwd_dev(h, pr.desc, pr.x0, None, pr.scal, pr.w, pr.prep, None, False, pr.x5, None, None)
            eoq.eoq_conv_fwd_dev(h, b.desc, b.x0, None, b.scal, b.w, b.prep, blk.shortcut, True, b.x5, b.x2, b.mask)
        last = self.blocks[-1].b
        n = fl.n
        eoq.eoq_aux_avgpool_sum(h, last.x5, n, self.hw, self.c_last, self.sums)
        # the head's own SGD step is not needed by the backward pass: it runs beside it
        eoq.eoq_aux_head(h, self.sums, n, self.c_last, self.hw, self.classes, self.W, self.bias, self.labels,
                         0.0 if overlap else self.head_lr, self.loss, self.dpooled, self.logits, self.head_ws)
        if overlap:
            self.sides[-1].wait_stream(main)
            with torch.cuda.stream(self.sides[-1]):
                eoq.eoq_aux_head_update(self.h_sides[-1], n, self.c_last, self.classes, self.W, self.bias, self.head_lr, self.head_ws)
        eoq.eoq_aux_head_error(h, self.dpooled, n, self.c_last, self.hw, self.e_head, self.e_head_exp, ws)

        side_no = [0]

        def wgrad_call(hh, u: UnitBuffers, b1_dev, wsp) -> None:
            if self.finish_together:
                u.b1_dev = b1_dev
                u.wgrad_parts = eoq.eoq_conv_wgrad_gemm(hh, u.desc, u.e3, u.e3_exp, u.x0, u.wgrad_ws)
            else:
                eoq.eoq_conv_wgrad_dev(hh, u.desc, u.e3, u.e3_exp, u.x0, b1_dev, u.g, u.g_exp, wsp)

        def wgrad(u: UnitBuffers, b1_dev) -> None:
            if overlap:
                k = side_no[0] % len(self.sides)
                side_no[0] += 1
                self.sides[k].wait_stream(main)
                with torch.cuda.stream(self.sides[k]):
                    wgrad_call(self.h_sides[k], u, b1_dev, self.workspace_sides[k])
            else:
                wgrad_call(h, u, b1_dev, ws)

        def finish(us) -> None:
            """b1 sums, slice sums and Q_g of the units whose GEMMs have been issued: a few launches for all of them,
            behind those GEMMs on a side stream (so that they run beside the rest of the backward chain)."""
            if not self.finish_together or not us:
                return
            args = ([u.desc for u in us], [u.e3 for u in us], [u.e3_exp for u in us], [u.b1_dev for u in us], [u.g for u in us],
                    [u.g_exp for u in us], [u.wgrad_ws for u in us], [u.wgrad_parts for u in us])
            if overlap:
                for side in self.sides[1:]:
                    self.sides[0].wait_stream(side)
                with torch.cuda.stream(self.sides[0]):
                    eoq.eoq_wgrad_finish(self.h_sides[0], *args)
            else:
                eoq.eoq_wgrad_finish(h, *args)

        e_out, e_exp = self.e_head, self.e_head_exp
        head_done = False   # the error head of this block's last unit already ran inside the join of the block behind it
        pending = []        # units whose weight-gradient GEMM is issued and not yet finished
        stage = None
        for i in reversed(range(len(self.blocks))):
            blk = self.blocks[i]
            a, b, pr = blk.a, blk.b, blk.proj
            if stage is not None and a.layer.name.split(".")[0] != stage:
                finish(pending)     # a stage of the network is through: its gradients are finished together
                pending = []
            stage = a.layer.name.split(".")[0]
            pending += [b, a] + ([pr] if pr else [])
            if not head_done:
                eoq.eoq_err_prescale_dev(h, e_out, e_exp, b.mask, b.x2, b.n_out, b.scal[1:2], b.e3, b.e3_exp, b.sum_e1, b.sum_e1x2)
            wgrad(b, b.scal[0:1])
            # error back through unit B; the error head of unit A rides on its Q_e
            eoq.eoq_conv_dgrad_head(h, b.desc, b.e3, b.e3_exp, b.w, b.e4, b.e4_exp, b.sum_e4, a.mask, None, a.scal[1:2], a.e3,
                                    a.e3_exp, a.sum_e1, None, ws)
            wgrad(a, a.scal[0:1])
            if pr:
                # the error entering the shortcut is e1 of unit B: e_out gated by unit B's ReLU mask
                eoq.eoq_err_prescale_dev(h, e_out, e_exp, b.mask, None, pr.n_out, self.c128, pr.e3, pr.e3_exp, pr.sum_e1, None)
                wgrad(pr, a.scal[0:1])
                eoq.eoq_conv_dgrad(h, pr.desc, pr.e3, pr.e3_exp, pr.w, pr.e4, pr.e4_exp, pr.sum_e4, None, ws)
                j_b, j_b_exp, j_mask = pr.e4, pr.e4_exp, None
            else:
                j_b, j_b_exp, j_mask = e_out, e_exp, b.mask
            # error back through unit A, joined with the shortcut's error; the joined error feeds the last unit of the
            # block in front (or the first layer when no pool sits between), whose error head rides on the join
            nxt = self.blocks[i - 1].b if i > 0 else (None if self.pool else stem)
            if nxt is not None:
                eoq.eoq_conv_dgrad_join_head(h, a.desc, a.e3, a.e3_exp, a.w, a.e4, a.e4_exp, a.sum_e4, j_b, j_b_exp, j_mask, blk.e_in,
                                             blk.e_in_exp, blk.sum_join, nxt.mask, nxt.x2, nxt.scal[1:2], nxt.e3, nxt.e3_exp,
                                             nxt.sum_e1, nxt.sum_e1x2 if nxt.x2 is not None else None, ws)
                head_done = True
            else:
                eoq.eoq_conv_dgrad_join_head(h, a.desc, a.e3, a.e3_exp, a.w, a.e4, a.e4_exp, a.sum_e4, j_b, j_b_exp, j_mask, blk.e_in,
                                             blk.e_in_exp, blk.sum_join, workspace=ws)
                head_done = False
            e_out, e_exp = blk.e_in, blk.e_in_exp
        finish(pending)
        if self.pool:
            k, s, p = self.pool
            # pool backward and the first layer's error head in one pair of kernels; the error between them (51 MB at
            # batch 64) is written only when a caller wants to look at it
            eoq.eoq_aux_maxpool_bwd_head(h, e_out, e_exp, self.pool_arg, fl.n, fl.ho, fl.wo, fl.c_out, k, s, p,
                                         self.stem_e0 if self.keep_pool_error else None, self.stem_e0_exp, stem.mask,
                                         stem.scal[1:2], stem.e3, stem.e3_exp, stem.sum_e1)
        elif not head_done:
            eoq.eoq_err_prescale_dev(h, e_out, e_exp, stem.mask, None, stem.n_out, stem.scal[1:2], stem.e3, stem.e3_exp, stem.sum_e1,
                                     None)
        wgrad(stem, None)
        finish([stem])
        if overlap:
            for side in self.sides:
                main.wait_stream(side)
        it = self.items
        eoq.eoq_aux_scalar_update(h, [i[0] for i in it], [i[1] for i in it], [i[2] for i in it], [i[3] for i in it],
                                  [i[4] for i in it], [i[5] for i in it], [i[6] for i in it], self.lr_mant, self.lr_exp,
                                  self.round_mode, self.seed, self.step_dev)
        eoq.eoq_update_dev(h, [u.w for u in self.units], [u.g for u in self.units], [u.g_exp for u in self.units],
                           self.lr_mant, self.lr_exp, self.round_mode, self.seed, self.step_dev)
        self.weight_prep()

    def capture(self, overlap: bool = True) -> None:
        """Records one step into a CUDA graph.  The warm-up step that precedes the capture is a real step: callers
        that need the state before it save and restore parameters, step counter and prepared weights."""
        cap = torch.cuda.Stream(device=self.dev, priority=-1)
        cap.wait_stream(torch.cuda.current_stream(self.dev))
        with torch.cuda.stream(cap):
            self.run(overlap)
        torch.cuda.synchronize(self.dev)
        before = self.launch_count()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph, stream=cap):
            self.run(overlap)
        torch.cuda.synchronize(self.dev)
        self.launches_per_step = self.launch_count() - before

    def replay(self) -> None:
        self.graph.replay()

    def host_image(self, seed: int) -> np.ndarray:
        f = self.units[0].layer
        return synth.normal_f32((f.n, f.h, f.w, self.image_channels), seed, 0)

    def result_tensors(self):
        """Small per-step results a caller would read back: the loss and the logits."""
        return [self.loss, self.logits]

    def time_conv_passes(self, replays: int = 5) -> dict:
        """Milliseconds per step of each convolution pass run alone, as TrainStep.time_conv_passes measures them."""
        h, ws = self.h, self.workspace
        s = torch.cuda.Stream(device=self.dev)

        def fwd():
            for u in self.units:
                eoq.eoq_conv_fwd_dev(h, u.desc, u.x0, self.image_exp if u.index == 0 else None, u.scal, u.w, u.prep,
                                     getattr(u, "shortcut", None), u.layer.relu, u.x5, u.x2, u.mask)

        def dgrad():
            for u in self.units:
                if u.e4 is not None:
                    eoq.eoq_conv_dgrad(h, u.desc, u.e3, u.e3_exp, u.w, u.e4, u.e4_exp, u.sum_e4, None, ws)

        def wgrad():
            for u in self.units:
                eoq.eoq_conv_wgrad_dev(h, u.desc, u.e3, u.e3_exp, u.x0, None if u.index == 0 else u.scal[0:1], u.g, u.g_exp, ws)

        def timed(fn) -> float:
            s.wait_stream(torch.cuda.current_stream(self.dev))
            with torch.cuda.stream(s):
                fn()
            torch.cuda.synchronize(self.dev)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                fn()
            torch.cuda.synchronize(self.dev)
            with torch.cuda.stream(s):
                for _ in range(2):
                    g.replay()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(s)
                for _ in range(replays):
                    g.replay()
                b.record(s)
            torch.cuda.synchronize(self.dev)
            return a.elapsed_time(b) / replays

        out = {"fwd": timed(fwd), "dgrad": timed(dgrad), "wgrad": timed(wgrad)}
        eoq.eoq_profile_gemm_only(h, True)
        try:
            out["dgrad_gemm"] = timed(dgrad)
            out["wgrad_gemm"] = timed(wgrad)
        finally:
            eoq.eoq_profile_gemm_only(h, False)
        return out

    def launch_count(self) -> int:
        return sum(eoq.eoq_launch_count(h) for h in [self.h] + self.h_sides)

    def status(self) -> int:
        st = 0
        for h in [self.h] + self.h_sides:
            st |= eoq.eoq_last_status(h)
        return st

    # ------------------------------------------------------------------ state (tests, trajectories)
    def parameters(self):
        return [u.w for u in self.units] + [u.scal for u in self.units] + [self.W, self.bias, self.step_dev]

    def save(self):
        return [p.clone() for p in self.parameters()]

    def restore(self, saved) -> None:
        for p, s in zip(self.parameters(), saved):
            p.copy_(s)
        self.weight_prep()

    def checksum(self) -> int:
        """A 64-bit checksum of every integer parameter (weights and scalars), cheap to compare step by step."""
        acc = 0
        for k, u in enumerate(self.units):
            w = u.w.view(torch.uint8).to(torch.int64)
            idx = torch.arange(w.numel(), device=w.device, dtype=torch.int64) % 65521 + 1
            acc = (acc * 1000003 + int((w.flatten() * idx).sum().item()) + 7 * k) % (1 << 61)
            acc = (acc * 1000003 + int(u.scal.to(torch.int64).mul(torch.tensor([3, 5, 7], device=w.device)).sum().item())) % (1 << 61)
        return acc

"""One training step's worth of hot-path calls over a workload (buffer plumbing only; all arithmetic is in libeoq).

For every quantized convolution layer of the network the step runs, through the C ABI:
  forward      eoq_conv_fwd     x0 -> x5 (+ x2 when gamma is trainable, + ReLU mask)
  error head   eoq_err_prescale e0, mask -> e3 (+ the sums behind g_b2 and g_gamma)
  dgrad        eoq_conv_dgrad   e3 -> e4          (not for the first layer)
  wgrad        eoq_conv_wgrad   e3, x0 -> g_w
and then one eoq_update over all weight tensors followed by one eoq_weight_prep (the b1 tables of the next
forward pass).  The network input is quantized by eoq_quantize_image at the start of every step.  The layer
scalars and the update's step counter live in device memory (the *_dev entry points), so a step captured into a
CUDA graph performs a new, correct step at every replay.  Layers are fed seeded synthetic tensors of the right shape and distribution
(post-ReLU codes as inputs, rounded-normal codes as incoming errors); pooling, the float classifier and the
residual error joins between layers are not part of this path.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

from . import eoq, synth
from .workloads import Layer, Workload, init_weight_f32



@dataclass
class Scalars:
    """Integer codes (p = -7) of the layer scalars used for every layer of a step."""
    b1_c: int = -2
    gamma_c: int = 118
    b2_c: int = 3


class LayerBuffers:
    def __init__(self, layer: Layer, dev, wmargin: int = 0):
        self.layer = layer
        self.wmargin = wmargin
        self.desc = eoq.conv_desc(layer.n, layer.h, layer.w, layer.c_in, layer.c_out, layer.k, layer.k, layer.stride, layer.pad,
                                  wmargin)
        i8, dev_ = torch.int8, dev
        out_shape = (layer.n, layer.ho, layer.wo, layer.c_out)
        in_shape = (layer.n, layer.h, layer.w, layer.c_in)
        self.x0 = torch.zeros((layer.n, layer.h, layer.w + 2 * wmargin, layer.c_in), dtype=i8, device=dev_)
        self.w = torch.empty((layer.c_out, layer.k, layer.k, layer.c_in), dtype=i8, device=dev_)
        self.x5 = torch.empty(out_shape, dtype=i8, device=dev_)
        self.x2 = torch.empty(out_shape, dtype=torch.int16, device=dev_) if layer.gamma_trainable else None
        n_out = int(np.prod(out_shape))
        self.mask = torch.empty((n_out + 7) // 8, dtype=torch.uint8, device=dev_) if layer.relu else None
        self.shortcut = torch.empty(out_shape, dtype=i8, device=dev_) if layer.shortcut else None
        self.e0 = torch.empty(out_shape, dtype=i8, device=dev_)
        self.e0_exp = torch.full((1,), -12, dtype=torch.int32, device=dev_)
        self.e3 = torch.empty(out_shape, dtype=i8, device=dev_)
        self.e3_exp = torch.zeros(1, dtype=torch.int32, device=dev_)
        self.e4 = torch.empty(in_shape, dtype=i8, device=dev_) if layer.has_dgrad else None
        self.e4_exp = torch.zeros(1, dtype=torch.int32, device=dev_)
        self.sum_e4 = torch.zeros(1, dtype=torch.int64, device=dev_)
        self.sum_e1 = torch.zeros(1, dtype=torch.int64, device=dev_)
        self.sum_e1x2 = torch.zeros(1, dtype=torch.int64, device=dev_)
        self.g = torch.empty_like(self.w)
        self.g_exp = torch.zeros(1, dtype=torch.int32, device=dev_)
        self.n_out = n_out
        # device-resident scalar codes {b1, gamma, b2} and what eoq_weight_prep derives from the weights
        self.scal = torch.zeros(3, dtype=torch.int32, device=dev_)
        self.prep = torch.empty(max(eoq.eoq_weight_prep_size(self.desc), 256), dtype=torch.uint8, device=dev_)


class TrainStep:
    """Allocates device buffers for a workload, fills them with seeded synthetic data, and runs steps."""

    def __init__(self, workload: Workload, handle: int, device: str = "cuda:0", seed: int = synth.BASE_SEED,
                 scalars: Optional[Scalars] = None, lr_mant: int = 1, lr_exp: int = -6, image_channels: int = 3,
                 side_streams: int = 2, round_mode: int = eoq.EOQ_ROUND_RNE):
        """round_mode: rounding of the update, EOQ_ROUND_RNE (the paper's R, Sec. 3.2.2) by default;
        EOQ_ROUND_STOCHASTIC is the labelled extension."""
        self.wl, self.h, self.dev = workload, handle, torch.device(device)
        self.sc = scalars or Scalars()
        self.lr_mant, self.lr_exp = lr_mant, lr_exp
        self.round_mode = round_mode
        self.step_dev = torch.zeros(1, dtype=torch.int64, device=self.dev)  # the update's step counter
        # the network input is stored with zero row margins so that a wide first-layer filter can fetch whole
        # filter rows (eoq_conv_desc_t::x_wmargin); every other layer input is dense
        # 5 = padding 3 plus an even distance, which the 8-channel layout needs for 16-byte aligned windows
        first_margin = 5 if workload.layers[0].k >= 5 else 0
        self.layers: List[LayerBuffers] = [LayerBuffers(l, self.dev, first_margin if i == 0 else 0)
                                           for i, l in enumerate(workload.layers)]
        ws = 256
        for lb in self.layers:
            for p in (eoq.EOQ_PASS_FWD, eoq.EOQ_PASS_DGRAD, eoq.EOQ_PASS_WGRAD):
                ws = max(ws, eoq.eoq_workspace_size(lb.desc, p))
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=self.dev)
        # further handles + workspaces: the weight-gradient chain of a layer can then run on a side stream next
        # to the layer's dgrad chain (a handle's reduction cells and a workspace serve one call at a time); the
        # chains of different layers are independent of each other, so they rotate over the side streams
        dev_index = self.dev.index if self.dev.index is not None else 0
        self.h_sides = [eoq.eoq_create(dev_index) for _ in range(side_streams)]
        self.workspace_sides = [torch.empty(ws, dtype=torch.uint8, device=self.dev) for _ in range(side_streams)]
        # the weight-gradient GEMMs of the side streams take half of the SMs each: two of them then run side by side
        # (and beside the helper kernels of the main chain) instead of one after the other
        half = torch.cuda.get_device_properties(self.dev).multi_processor_count // 2
        for hs in self.h_sides:
            eoq.eoq_set_gemm_ctas(hs, half)
        self.sides = [torch.cuda.Stream(device=self.dev) for _ in range(side_streams)]
        self.graph = None
        first = workload.layers[0]
        self.image_channels = image_channels
        self.image_pixels = first.n * first.h * first.w
        self.image = torch.empty((first.n, first.h, first.w, image_channels), dtype=torch.float32, device=self.dev)
        self.image_exp = torch.zeros(1, dtype=torch.int32, device=self.dev)
        self._fill(seed)

    # ------------------------------------------------------------------ synthetic data (host side, numpy)
    def host_image(self, seed: int) -> np.ndarray:
        f = self.wl.layers[0]
        return synth.normal_f32((f.n, f.h, f.w, self.image_channels), seed, 0)

    def _fill(self, seed: int) -> None:
        self.image.copy_(torch.from_numpy(self.host_image(seed)))
        pools = {}

        def pooled(kind, shape, stream):
            key = (kind, tuple(shape))
            if key not in pools:
                gen = {"relu": synth.relu_codes, "err": synth.normal_codes, "uni": synth.int8_uniform}[kind]
                pools[key] = torch.from_numpy(gen(shape, seed, stream))
            return pools[key]

        for i, lb in enumerate(self.layers):
            l = lb.layer
            if i > 0:
                lb.x0.copy_(pooled("relu", lb.x0.shape, 1))
            lb.e0.copy_(pooled("err", lb.e0.shape, 2))
            if lb.shortcut is not None:
                lb.shortcut.copy_(pooled("relu", lb.shortcut.shape, 3))
            wf = init_weight_f32(l, self.wl, synth.normal_f64(tuple(lb.w.shape), seed, 100 + i))
            wf_d = torch.from_numpy(wf).to(self.dev)
            eoq.eoq_quantize(self.h, eoq.EOQ_CQ, wf_d, True, None, wf_d.numel(), lb.w)  # Q_w, once at initialisation
        self.set_scalars(self.sc)
        self.weight_prep()
        torch.cuda.synchronize(self.dev)

    def layer_scalars(self, i: int):
        """(b1, gamma, b2) codes of layer i under the step's Scalars: no bias in front of the first layer, gamma
        fixed at 1 (code 128) where it is not trainable, no b2 on a projection shortcut."""
        l = self.layers[i].layer
        sc = self.sc
        return (0 if i == 0 else sc.b1_c, sc.gamma_c if l.gamma_trainable else 128, sc.b2_c if l.relu else 0)

    def set_scalars(self, sc: Scalars) -> None:
        self.sc = sc
        for i, lb in enumerate(self.layers):
            lb.scal.copy_(torch.tensor(self.layer_scalars(i), dtype=torch.int32))

    def weight_prep(self) -> None:
        eoq.eoq_weight_prep(self.h, [lb.desc for lb in self.layers], [lb.w for lb in self.layers],
                            [lb.prep for lb in self.layers])

    # ------------------------------------------------------------------ one step
    def run(self, overlap: bool = False) -> None:
        """One step on the current stream.  overlap=True forks every layer's weight-gradient chain to a side
        stream (it only needs the layer's e3 and x0) and joins before the update."""
        h, sc, ws = self.h, self.sc, self.workspace
        main = torch.cuda.current_stream(self.dev)
        first = self.layers[0]
        fl = first.layer
        eoq.eoq_quantize_image(h, self.image, fl.n, fl.h, fl.w, self.image_channels, fl.c_in, first.wmargin, first.x0,
                               self.image_exp)
        for i, lb in enumerate(self.layers):
            l = lb.layer
            eoq.eoq_conv_fwd_dev(h, lb.desc, lb.x0, self.image_exp if i == 0 else None, lb.scal, lb.w, lb.prep, lb.shortcut,
                                 l.relu, lb.x5, lb.x2, lb.mask)
        for i in range(len(self.layers) - 1, -1, -1):
            lb = self.layers[i]
            l = lb.layer
            b1_dev = None if i == 0 else lb.scal[0:1]
            eoq.eoq_err_prescale_dev(h, lb.e0, lb.e0_exp, lb.mask, lb.x2, lb.n_out, lb.scal[1:2], lb.e3, lb.e3_exp, lb.sum_e1,
                                     lb.sum_e1x2 if lb.x2 is not None else None)
            if overlap:
                k = i % len(self.sides)
                self.sides[k].wait_stream(main)
                with torch.cuda.stream(self.sides[k]):
                    eoq.eoq_conv_wgrad_dev(self.h_sides[k], lb.desc, lb.e3, lb.e3_exp, lb.x0, b1_dev, lb.g, lb.g_exp,
                                           self.workspace_sides[k])
            if l.has_dgrad:
                eoq.eoq_conv_dgrad(h, lb.desc, lb.e3, lb.e3_exp, lb.w, lb.e4, lb.e4_exp, lb.sum_e4, None, ws)
            if not overlap:
                eoq.eoq_conv_wgrad_dev(h, lb.desc, lb.e3, lb.e3_exp, lb.x0, b1_dev, lb.g, lb.g_exp, ws)
        if overlap:
            for side in self.sides:
                main.wait_stream(side)
        eoq.eoq_update_dev(h, [lb.w for lb in self.layers], [lb.g for lb in self.layers], [lb.g_exp for lb in self.layers],
                           self.lr_mant, self.lr_exp, self.round_mode, synth.BASE_SEED, self.step_dev)
        self.weight_prep()  # the tables the next forward pass reads

    def capture(self, overlap: bool = True) -> None:
        """Records one step into a CUDA graph (after an eager warm-up step on the capture stream).  Scalars and the
        update's step counter are read from device memory, so every replay is the next step of the run."""
        # the capture stream carries the chain every layer waits on (error head -> dgrad -> next error head): it gets
        # the higher priority, so that its kernels are placed before the side streams' weight-gradient work
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

    def time_conv_passes(self, replays: int = 5) -> dict:
        """Milliseconds per step of each convolution pass run alone: the calls of one pass over all layers are recorded
        back to back into their own CUDA graph (one stream) and a run of replays is timed with CUDA events on the
        launching stream.  fwd: the forward GEMM launches (nothing else runs in a forward call); dgrad / wgrad: the
        whole calls; dgrad_gemm / wgrad_gemm: their GEMM kernels only (eoq_profile_gemm_only)."""
        h, ws = self.h, self.workspace
        s = torch.cuda.Stream(device=self.dev)

        def fwd():
            for i, lb in enumerate(self.layers):
                eoq.eoq_conv_fwd_dev(h, lb.desc, lb.x0, self.image_exp if i == 0 else None, lb.scal, lb.w, lb.prep,
                                     lb.shortcut, lb.layer.relu, lb.x5, lb.x2, lb.mask)

        def dgrad():
            for lb in self.layers:
                if lb.layer.has_dgrad:
                    eoq.eoq_conv_dgrad(h, lb.desc, lb.e3, lb.e3_exp, lb.w, lb.e4, lb.e4_exp, lb.sum_e4, None, ws)

        def wgrad():
            for i, lb in enumerate(self.layers):
                eoq.eoq_conv_wgrad_dev(h, lb.desc, lb.e3, lb.e3_exp, lb.x0, None if i == 0 else lb.scal[0:1], lb.g, lb.g_exp, ws)

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

    def replay(self) -> None:
        self.graph.replay()

    def launch_count(self) -> int:
        return sum(eoq.eoq_launch_count(h) for h in [self.h] + self.h_sides)

    def status(self) -> int:
        st = 0
        for h in [self.h] + self.h_sides:
            st |= eoq.eoq_last_status(h)
        return st

    def result_tensors(self):
        """Small per-step results a caller would read back: every gradient exponent and the last activation."""
        return [lb.g_exp for lb in self.layers] + [self.layers[-1].x5]

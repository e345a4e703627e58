#!/usr/bin/env python
"""Benchmark of the EOQ int8 convolution training path (arXiv 2105.13890) on B200.

One step = one closed-loop int8 training step of Fixup ResNet-18 (batch 64, 224x224) on synthetic images and
labels: input quantizer, every quantized convolution unit forward (chained, with max-pooling and shortcuts), global
average pooling and the floating-point last layer, then back: per unit error head + dgrad + wgrad with the error joins
at the block inputs, and the 8-bit update of all weights plus the update of the scalars.  --independent times the
same convolution units fed independent synthetic tensors instead (no glue between them; also the only mode for
the bottleneck and single-layer workloads).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet18|resnet20|resnet50|single] [--batch B]
  python bench.py --impl reference ...     # the CPU oracle on host cores, same metric, bounded sample per step
  python bench.py --probe mma_i8           # INT8 tensor-pipe denominators: own tcgen05.mma issue-rate probe + a library int8 matmul

With --gpus N > 1 and no launcher environment the script starts N ranks of itself (one per GPU, rendezvous on
127.0.0.1); under torchrun it is one of the ranks.  Every rank runs the whole per-GPU workload (replicas), rank 0
prints the line.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "int8 conv TOPS per train step (fwd+dgrad+wgrad) and img/s, % of INT8 roofline"
INT8_OVER_BF16 = 2.0  # nominal dense ratio (4.5 / 2.25 PFLOP/s)
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the implicit-GEMM kernels, from an ncu capture of the
# present kernels (profiles/); None while no capture of the current kernels exists
IGEMM_DRAM_BYTES_PER_LAUNCH = {}
NOMINAL_INT8_TOPS = 4500.0  # public dense figure, context only


def peaks():
    """Measured denominators (generated file) or the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"],
                "bf16_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------------------------- clocks

class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc, self.lines = None, []
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def window(self, t0, t1):
        return [l for (t, l) in self.lines if t0 <= t <= t1]

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    @staticmethod
    def summarize(lines):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------- CPU oracle arm

def oracle_step(wl, seed, scal):
    """One step of the same path on the CPU oracle, as it stands.  Returns seconds."""
    import numpy as np

    import oracle
    from oracle import ConvDesc
    from paper_2105_13890_b200 import synth

    b1_c, gamma_c, b2_c = scal
    # inputs first (not timed: the GPU arm's inputs are resident before its timed region too)
    data = []
    first = wl.layers[0]
    image = synth.normal_f32((first.n, first.h, first.w, 3), seed, 0)
    for i, l in enumerate(wl.layers):
        d = ConvDesc(l.n, l.h, l.w, l.c_in, l.c_out, l.k, l.k, l.stride, l.pad)
        x0 = synth.relu_codes((l.n, l.h, l.w, l.c_in), seed, 1) if i else None
        e0 = synth.normal_codes((l.n, l.ho, l.wo, l.c_out), seed, 2)
        sc = synth.relu_codes((l.n, l.ho, l.wo, l.c_out), seed, 3) if l.shortcut else None
        wf = oracle.fixup_weights_f32(synth.normal_f64((l.c_out, l.k, l.k, l.c_in), seed, 100 + i),
                                      l.c_in_true * l.k * l.k, wl.L, wl.m, l.in_branch)
        wf[..., l.c_in_true:] = 0.0
        data.append((l, d, x0, e0, sc, oracle.q_w(wf)))
    t0 = time.perf_counter()
    img = np.zeros((first.n, first.h, first.w, first.c_in), dtype=np.float32)
    img[..., :3] = image
    codes, p_in, _ = oracle.quantize_f32(oracle.MODE_SQ, img)
    saved = []
    for i, (l, d, x0, e0, sc, w) in enumerate(data):
        if i == 0:
            x0 = codes.astype(np.int8)
        gamma = gamma_c if l.gamma_trainable else 128
        fwd = oracle.layer_forward(d, x0, 0 if i == 0 else b1_c, w, gamma, b2_c if l.relu else 0, sc, l.relu,
                                   x_exp=p_in if i == 0 else -7)
        saved.append((x0, fwd))
    grads = []
    for i in range(len(data) - 1, -1, -1):
        l, d, _, e0, sc, w = data[i]
        x0, fwd = saved[i]
        gamma = gamma_c if l.gamma_trainable else 128
        mask = fwd["mask"] if l.relu else np.ones_like(fwd["mask"])
        e3, p3, s1, s2, _ = oracle.err_prescale(e0, -12, mask, fwd["x2"] if l.gamma_trainable else None, gamma)
        if l.has_dgrad:
            oracle.sq_int(oracle.conv_dgrad_acc(d, e3, w), p3 - 7)
        g, pg, _ = oracle.sq_int(oracle.conv_wgrad_acc(d, e3, x0, 0 if i == 0 else b1_c), p3 - 7)
        grads.append((i, g.astype(np.int8), pg))
    for i, g, pg in grads:
        oracle.update(data[i][5], g, pg, 1, -6, stochastic=False)
    return time.perf_counter() - t0


CHAINED = {"resnet18": ("resnet18", 1000, (3, 2, 1)), "resnet34": ("resnet34", 1000, (3, 2, 1)),
           "resnet20": ("resnet20", 10, None), "resnet110": ("resnet110", 10, None)}


def oracle_chain_step(name, batch, seed):
    """One closed-loop training step of the same network on the CPU oracle, as it stands.  Returns seconds."""
    import oracle
    from oracle import network as N
    from paper_2105_13890_b200 import synth

    oname, classes, _ = CHAINED[name]
    net = getattr(N, oname)(batch)
    N.init(net, lambda s, st: synth.normal_f64(s, seed, st), lambda s, st: synth.normal_f32(s, seed, st), b1=-2, gamma=118, b2=3)
    f = net.units[0].d
    img = synth.normal_f32((f.n, f.h, f.w, 3), seed, 0)
    labels = synth.labels(f.n, classes, seed, 1)
    t0 = time.perf_counter()
    N.train_step(net, img, labels, 1, -8, 2.0 ** -6, keep=False)
    return time.perf_counter() - t0


def cpu_step_seconds(args, wl):
    """The oracle's step for the mode the GPU arm times."""
    if args.workload in CHAINED and not args.independent:
        return oracle_chain_step(args.workload, wl.batch, 1)
    return oracle_step(wl, 1, (-2, 118, 3))


def run_reference(args):
    """--impl reference: the oracle timed on the host cores, each step a bounded sample (small batch) of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2105_13890_b200 import workloads

    oracle.build()
    sample_batch = args.ref_arm_batch
    wl = workloads.get(args.workload, sample_batch)
    full = workloads.get(args.workload, args.batch)
    cores = os.cpu_count() or 1
    for _ in range(args.warmup):
        cpu_step_seconds(args, wl)
    secs = [cpu_step_seconds(args, wl) for _ in range(args.steps)]
    t = sum(secs) / len(secs)
    tops = wl.total_ops / t / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": tops, "unit": "TOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "img_per_s": wl.batch / t,
        "config": {"workload": full.name, "sample": f"batch {sample_batch} of {full.batch} per step, all layers",
                   "step": "independent layer units" if (args.independent or args.workload not in CHAINED) else "closed loop"},
        "cpu_baseline": {"value": tops, "unit": "TOPS", "cores": cores, "kind": "oracle",
                         "sample": f"{wl.name}: every layer of the workload at batch {sample_batch}"},
        "e2e": {"value": tops, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- GPU arm

def bandwidth_bytes(wl, chained=False):
    """Algorithmic bytes per step of the bandwidth-bound kernel groups (what the method itself must move).
    In the closed-loop step most error heads ride on the kernel that produces their input error: the head of a block's
    first unit on the Q_e pass behind the second unit's dgrad (its bytes are counted there), the others on joins and the
    pool's backward (glue, not listed); only the last block's and the projection shortcuts' heads run on their own."""
    head = dq = fin = upd = 0
    last_b = max((i for i, l in enumerate(wl.layers) if l.name.endswith(".b")), default=-1)
    for i, l in enumerate(wl.layers):
        n_out = l.n * l.ho * l.wo * l.c_out
        own = n_out * (1 + 1 + 0.125 + (2 if l.gamma_trainable else 0))    # e0 in, e3 out, mask, x2 for g_gamma
        if not chained or l.name.endswith(".proj") or i == last_b:
            head += own
        elif l.name.endswith(".a"):
            dq += n_out * (1 + 0.125)                                       # e3 out and mask bits, on the Q_e pass of unit B
        if l.has_dgrad:
            dq += l.n * l.h * l.w * l.c_in * (4 + 1)                        # exact int32 sums in, e4 codes out
        fin += l.weight_elems * (4 + 1)                                     # exact sums in, g codes out
        upd += l.weight_elems * 3                                           # g in, w in, w out
    f = wl.layers[0]
    inq = f.n * f.h * f.w * (3 * 4 * 2 + f.c_in)                            # fp32 image read twice (max, code), codes out
    return {"err_head": head, "dgrad_aux": dq, "wgrad_aux": fin, "update": upd, "input_quantizer": inq}


def run_gpu(args):
    import torch

    from paper_2105_13890_b200 import eoq, ranks, workloads
    from paper_2105_13890_b200.chain import ChainedStep
    from paper_2105_13890_b200.step import Scalars, TrainStep

    world, rank, local = ranks.world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    ranks.init("nccl", torch.device("cuda", local))
    barrier = ranks.barrier

    wl = workloads.get(args.workload, args.batch)
    handle = eoq.eoq_create(local)
    round_mode = eoq.EOQ_ROUND_STOCHASTIC if args.stochastic else eoq.EOQ_ROUND_RNE
    chained = args.workload in CHAINED and not args.independent
    if chained:
        _, classes, pool = CHAINED[args.workload]
        step = ChainedStep(wl, handle, f"cuda:{local}", scalars=Scalars(), lr_mant=1, lr_exp=-8, classes=classes, pool=pool,
                           round_mode=round_mode)
        step.image.copy_(torch.from_numpy(step.host_image(777)))
        step.labels.copy_(torch.from_numpy(__import__("numpy").arange(wl.batch, dtype="int32") % classes))
    else:
        step = TrainStep(wl, handle, f"cuda:{local}", scalars=Scalars(), round_mode=round_mode)
    stream = torch.cuda.current_stream()

    # One step = one replay of a CUDA graph of the whole path (the weight-gradient chain of each layer on a side
    # stream next to its dgrad chain); --eager launches call by call on one stream instead.
    if args.eager:
        do_step = step.run
    else:
        step.capture(overlap=True)
        do_step = step.replay
    for _ in range(args.warmup):
        do_step()
    barrier()
    status = step.status()

    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.3)
    # ---- timed region: K steps, inputs resident
    l0 = step.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        do_step()
    ev1.record(stream)
    barrier()
    t_wall1 = time.time()
    ms = ev0.elapsed_time(ev1)
    launches = step.launch_count() - l0
    if not args.eager:
        launches = step.launches_per_step * args.steps  # graph replays do not pass through the host-side counter
    status |= step.status()
    if args.step_only:
        # for a launch list under a profiler: the steps above are all that runs (no end-to-end, per-kernel or per-kind pass)
        if rank == 0:
            print(json.dumps({"metric": METRIC, "step_only": True, "ms_per_step": ms / args.steps, "steps": args.steps,
                              "warmup": args.warmup, "gpu_launches": int(launches), "device_status": int(status),
                              "config": {"workload": wl.name}}), flush=True)
        if sampler:
            sampler.stop()
        eoq.eoq_destroy(handle)
        ranks.finish()
        return

    # ---- end to end: host image in (pinned), results out, every step
    host_img = torch.from_numpy(step.host_image(12345)).pin_memory()
    results = step.result_tensors()
    host_out = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in results]
    h2d = host_img.numel() * host_img.element_size()
    d2h = sum(t.numel() * t.element_size() for t in results)
    # The image of step k + 1 travels host -> device on a copy stream while step k computes (two staging buffers,
    # as a data loader would); the step itself starts with a device-to-device copy of its staged image.  Every
    # step's host -> device copy and its device -> host read lie inside the timed region.
    copy_stream = torch.cuda.Stream()
    staging = [torch.empty_like(step.image) for _ in range(2)]
    staged = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]

    def stage(k):
        with torch.cuda.stream(copy_stream):
            if k >= 2:
                copy_stream.wait_event(consumed[k % 2])  # the step that read this buffer last has taken its copy
            staging[k % 2].copy_(host_img, non_blocking=True)
            staged[k % 2].record(copy_stream)

    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    copy_stream.wait_event(e0)
    stage(0)
    for k in range(args.steps):
        if k + 1 < args.steps:
            stage(k + 1)
        stream.wait_event(staged[k % 2])
        step.image.copy_(staging[k % 2], non_blocking=True)
        consumed[k % 2].record(stream)
        do_step()
        for src, dst in zip(results, host_out):
            dst.copy_(src, non_blocking=True)
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)

    # ---- the convolution kernels alone, replayed back to back from their own graphs (forward: one GEMM launch per
    # layer; dgrad: GEMM + Q_e; wgrad: the whole weight-gradient call), CUDA events around a run of replays on the
    # launching stream.  This is the launch duration the roofline figure uses: event brackets around single launches
    # add several microseconds of event overhead to kernels that last 10 to 30.
    conv_ms = step.time_conv_passes(replays=max(3, min(10, args.steps)))

    # ---- per-kind timing (events around each launch, eager, one stream)
    # Each eager step is queued behind a few milliseconds of device-side delay, so that the host has issued the
    # whole step before the device starts it: the events then bracket device time only, not host launch gaps.
    # The library keeps a bounded number of event pairs per profiling session (8192): profile as many steps as fit.
    prof_steps = max(1, min(args.steps, 8000 // max(1, int(launches) // max(1, args.steps))))
    eoq.eoq_profile_start(handle)
    for _ in range(prof_steps):
        torch.cuda._sleep(12_000_000)
        step.run()
    prof_n, prof_ms = eoq.eoq_profile_stop(handle)
    # the tensor pipe's own INT8 figure, measured on the spot (issue-rate probe, N = 256, about ten milliseconds)
    probe_tops, _ = eoq.eoq_probe_mma_i8(handle, 256, 2048, 10)
    t_wall2 = time.time()
    # clocks while the GPU was under this load: the timed steps first, the whole loaded span if that is too short
    clocks = None
    if sampler:
        lines = sampler.window(t_wall0, t_wall1)
        if len(lines) < 5:
            lines = sampler.window(t_wall0, t_wall2)
        clocks = ClockSampler.summarize(lines)
        sampler.stop()

    ms, ms_e2e = ranks.max_over_ranks([ms, ms_e2e], device=f"cuda:{local}")

    if rank == 0:
        pk = peaks()
        ops_step = wl.total_ops
        sec = ms / 1e3 / args.steps
        tops = ranks.whole_job_rate(ops_step, args.steps, ms, world) / 1e12
        tops_e2e = ranks.whole_job_rate(ops_step, args.steps, ms_e2e, world) / 1e12
        # the clocks stay at their maximum over the step (see "clocks"), so the burst bf16 figure is the denominator
        int8_peak = pk["bf16_burst"] * INT8_OVER_BF16
        fwd_ops = sum(2 * l.macs for l in wl.layers)
        dgrad_ops = sum(2 * l.macs for l in wl.layers if l.has_dgrad)
        n_fwd = len(wl.layers)
        n_dgrad = sum(1 for l in wl.layers if l.has_dgrad)
        igemm_ms = conv_ms["fwd"] + conv_ms["dgrad_gemm"]
        achieved = (fwd_ops + dgrad_ops) / (igemm_ms / 1e3) / 1e12
        names = eoq.EOQ_PROF_NAMES
        by_kind = {name: prof_ms[i] / prof_steps for i, name in enumerate(names)}
        bw = {}
        for kind, nbytes in bandwidth_bytes(wl, chained).items():
            t_ms = by_kind.get(kind, 0.0)
            gbs = nbytes / (t_ms / 1e3) / 1e9 if t_ms > 0 else None
            bw[kind] = {"algorithmic_bytes": nbytes, "ms": t_ms, "gbs": gbs, "frac_of_hbm": gbs / pk["hbm_gbs"] if gbs else None}
        line = {
            "metric": METRIC, "value": tops, "unit": "TOPS", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "img_per_s": world * wl.batch / sec,
            "pct_of_int8_peak": 100.0 * tops / world / int8_peak,
            "config": {"workload": wl.name, "layers": len(wl.layers), "global_batch": world * wl.batch,
                       "gop_per_step": ops_step / 1e9, "l2": "working set larger than L2; no flush between steps",
                       "step": "closed loop: units chained, pooling, float head, error joins, scalar updates" if chained
                               else "independent layer units on synthetic tensors",
                       "scalars": "b1=-2 gamma=118 b2=3 codes at the start, device-resident",
                       "update": "stochastic rounding (extension)" if args.stochastic else "round to nearest even (Sec. 3.2.2)",
                       "parallelism": f"replicas x{world}",
                       "launch": "eager, one stream" if args.eager else "CUDA graph replay, wgrad chains on two side streams"},
            "clocks": clocks,
            "e2e": {"value": tops_e2e, "unit": "TOPS", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": int(launches),
            "device_status": int(status),
            "roofline": {
                "kernel": "igemm_kernel + igemm_patch_kernel (forward + dgrad implicit GEMM, tcgen05 kind::i8)",
                "bound": "tensor", "achieved": achieved, "peak": int8_peak, "unit": "TOPS", "frac": achieved / int8_peak,
                "traffic": IGEMM_DRAM_BYTES_PER_LAUNCH.get(wl.name),
                "peak_source": f"{pk['source']} burst bf16 {pk['bf16_burst']} TFLOP/s x {INT8_OVER_BF16} (nominal int8:bf16)",
                "launches": n_fwd + n_dgrad, "avg_launch_ms": igemm_ms / (n_fwd + n_dgrad),
                "timing": "graph replay of the launches back to back, CUDA events around the run",
                "frac_of_nominal_4500": achieved / NOMINAL_INT8_TOPS,
                "frac_of_sustained_bf16_x2": achieved / (pk["bf16_sustained"] * INT8_OVER_BF16),
                "mma_i8_probe_tops": probe_tops, "frac_of_mma_i8_probe": achieved / probe_tops,
            },
            "kernels": {
                "igemm_fwd": {"launches": n_fwd, "ms": conv_ms["fwd"], "tops": fwd_ops / (conv_ms["fwd"] / 1e3) / 1e12},
                "igemm_dgrad": {"launches": n_dgrad, "ms": conv_ms["dgrad_gemm"],
                                "tops": dgrad_ops / (conv_ms["dgrad_gemm"] / 1e3) / 1e12},
                "dgrad_with_Qe": {"ms": conv_ms["dgrad"], "tops": dgrad_ops / (conv_ms["dgrad"] / 1e3) / 1e12},
                "wgrad": {"launches": n_fwd, "ms": conv_ms["wgrad_gemm"], "tops": fwd_ops / (conv_ms["wgrad_gemm"] / 1e3) / 1e12},
                "wgrad_with_Qg": {"ms": conv_ms["wgrad"], "tops": fwd_ops / (conv_ms["wgrad"] / 1e3) / 1e12},
            },
            "bandwidth_kernels": bw,
            "ms_per_step_by_kind": by_kind,
            "profiled_steps": prof_steps,
        }
        if args.int8_peaks:
            # the two measured INT8 figures next to the denominator in use (see --probe)
            line["int8_peaks"] = json.loads(args.int8_peaks)
            for k, v in line["int8_peaks"].items():
                if isinstance(v, (int, float)) and v > 0 and k.endswith("_tops"):
                    line["roofline"][f"frac_of_{k}"] = achieved / v
        if world == 1 and not args.no_cpu_baseline:
            import oracle

            oracle.build()
            small = workloads.get(args.workload, args.ref_batch if args.ref_batch else wl.batch)
            secs = cpu_step_seconds(args, small)
            line["cpu_baseline"] = {"value": small.total_ops / secs / 1e12, "unit": "TOPS", "cores": os.cpu_count(),
                                    "kind": "oracle", "seconds": secs,
                                    "sample": f"{small.name}: every layer of the workload at batch {small.batch}, one step"}
        print(json.dumps(line), flush=True)
    eoq.eoq_destroy(handle)
    ranks.finish()


# ----------------------------------------------------------------------------------------------- INT8 peak probe

def run_probe(args):
    """INT8 tensor-pipe figures to hold the roofline against: the library's own tcgen05.mma kind::i8 issue-rate probe
    (operands in shared memory, every SM) and, as an independent library figure, an int8 matmul through torch."""
    import torch

    from paper_2105_13890_b200 import eoq

    if not torch.cuda.is_available():
        raise SystemExit("bench.py --probe needs a CUDA device")
    h = eoq.eoq_create(0)
    out = {"probe": "mma_i8", "unit": "TOPS"}
    sampler = ClockSampler(0)
    t0 = time.time()
    for n in (256, 128, 64):
        burst, cyc = eoq.eoq_probe_mma_i8(h, n, 2048, 10)           # ~1 ms per launch
        t_end = time.time() + args.probe_seconds
        sustained = []
        while time.time() < t_end:
            sustained.append(eoq.eoq_probe_mma_i8(h, n, 8192, 50)[0])
        out[f"mma_i8_n{n}_burst_tops"] = burst
        out[f"mma_i8_n{n}_sustained_tops"] = sum(sustained[len(sustained) // 2:]) / max(1, len(sustained) - len(sustained) // 2)
        out[f"mma_i8_n{n}_cycles_per_mma"] = cyc
    assert eoq.eoq_last_status(h) == 0
    # library int8 matmul, 8192^3 (measurement only; never on the layer's path)
    try:
        a = torch.randint(-8, 8, (8192, 8192), dtype=torch.int8, device="cuda")
        b = torch.randint(-8, 8, (8192, 8192), dtype=torch.int8, device="cuda").t()
        for _ in range(3):
            torch._int_mm(a, b)
        best = None
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch._int_mm(a, b)
            e1.record()
            torch.cuda.synchronize()
            t = e0.elapsed_time(e1)
            best = t if best is None or t < best else best
        out["library_int8_matmul_8192_tops"] = 2 * 8192 ** 3 / (best / 1e3) / 1e12
    except Exception as ex:  # the library routine is optional: report why it is absent
        out["library_int8_matmul_8192_tops"] = None
        out["library_int8_matmul_error"] = str(ex)[:200]
    out["clocks"] = ClockSampler.summarize(sampler.window(t0, time.time()))
    sampler.stop()
    pk = peaks()
    out["denominator_in_bench_line"] = pk["bf16_burst"] * INT8_OVER_BF16
    out["nominal_tops"] = NOMINAL_INT8_TOPS
    eoq.eoq_destroy(h)
    print(json.dumps(out), flush=True)


# ----------------------------------------------------------------------------------------------- BN comparison

def run_bn_compare(args):
    """--probe bn_vs_fixup: the paper's second claim restated on this device (Sec. 5.3): on the same int8 convolutions of
    Fixup ResNet-18, the fused scale-and-bias epilogue of EOQ against training-mode batch normalisation behind the
    convolution (eoq_bn_fwd / eoq_bn_bwd: two extra passes over the exact sums forward, two more backward, then Q_e).
    Each variant is replayed from a CUDA graph of ten copies of its calls; times are per call."""
    import torch

    from paper_2105_13890_b200 import eoq, workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py --probe needs a CUDA device")
    dev = "cuda:0"
    h = eoq.eoq_create(0)
    wl = workloads.get("resnet18", args.batch)
    picks = [l for l in wl.layers if l.name in ("layer1.0.a", "layer2.1.a", "layer3.1.a", "layer4.1.a")]
    g = torch.Generator(device=dev)
    g.manual_seed(4242)

    def time_calls(fn, copies=10, replays=5):
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            fn()
            fn()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            for _ in range(copies):
                fn()
        torch.cuda.synchronize()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(replays):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (copies * replays) * 1e3   # microseconds per call

    rows = []
    for l in picks:
        d = eoq.conv_desc(l.n, l.h, l.w, l.c_in, l.c_out, l.k, l.k, l.stride, l.pad)
        shape = (l.n, l.ho, l.wo, l.c_out)
        n_out = l.n * l.ho * l.wo * l.c_out
        x0 = torch.randint(0, 100, (l.n, l.h, l.w, l.c_in), dtype=torch.int8, device=dev, generator=g)
        x0 = torch.where(torch.rand(x0.shape, device=dev, generator=g) < 0.5, torch.zeros_like(x0), x0)
        w = torch.randint(-6, 7, (l.c_out, l.k, l.k, l.c_in), dtype=torch.int8, device=dev, generator=g)
        e0 = torch.randint(-90, 91, shape, dtype=torch.int8, device=dev, generator=g)
        e0_exp = torch.full((1,), -12, dtype=torch.int32, device=dev)
        x5, x2 = torch.zeros(shape, dtype=torch.int8, device=dev), torch.zeros(shape, dtype=torch.int16, device=dev)
        mask = torch.zeros((n_out + 7) // 8, dtype=torch.uint8, device=dev)
        acc = torch.zeros(shape, dtype=torch.int32, device=dev)
        ws = torch.empty(max(eoq.eoq_workspace_size(d, eoq.EOQ_PASS_FWD), 256), dtype=torch.uint8, device=dev)
        e3, e3_exp = torch.zeros(shape, dtype=torch.int8, device=dev), torch.zeros(1, dtype=torch.int32, device=dev)
        s1, s2 = torch.zeros(1, dtype=torch.int64, device=dev), torch.zeros(1, dtype=torch.int64, device=dev)
        bn_ws = torch.zeros(eoq.eoq_bn_workspace_size(l.c_out), dtype=torch.uint8, device=dev)
        gamma_f = torch.ones(l.c_out, dtype=torch.float32, device=dev)
        beta_f = torch.zeros(l.c_out, dtype=torch.float32, device=dev)
        da = torch.zeros(shape, dtype=torch.float32, device=dev)
        dg, db = torch.zeros(l.c_out, dtype=torch.float32, device=dev), torch.zeros(l.c_out, dtype=torch.float32, device=dev)
        pixels = l.n * l.ho * l.wo

        def fwd_eoq():
            eoq.eoq_conv_fwd(h, d, x0, None, 0, w, 118, 3, None, True, x5, x2, mask, None, ws)

        def fwd_conv_dump():
            eoq.eoq_conv_fwd(h, d, x0, None, 0, w, 118, 3, None, True, x5, x2, mask, acc, ws)

        def fwd_bn():
            eoq.eoq_bn_fwd(h, acc, -14, pixels, l.c_out, gamma_f, beta_f, 1e-5, x5, mask, bn_ws)

        def bwd_eoq():
            eoq.eoq_err_prescale(h, e0, e0_exp, mask, x2, n_out, 118, e3, e3_exp, s1, s2)

        def bwd_bn():
            eoq.eoq_bn_bwd(h, e0, e0_exp, mask, acc, -14, pixels, l.c_out, gamma_f, bn_ws, da, dg, db)
            eoq.eoq_quantize(h, eoq.EOQ_SQ, da, True, None, n_out, e3, e3_exp)

        t = {"fwd_eoq_conv_fused_us": time_calls(fwd_eoq), "fwd_conv_with_sum_dump_us": time_calls(fwd_conv_dump),
             "fwd_bn_passes_us": time_calls(fwd_bn), "bwd_eoq_error_head_us": time_calls(bwd_eoq),
             "bwd_bn_passes_and_Qe_us": time_calls(bwd_bn)}
        # BN forward = convolution that writes its exact sums + the BN passes; the dump run here also computes the fused
        # epilogue, so the lower figure replaces it by the fused convolution's own time
        t["fwd_bn_total_us"] = [t["fwd_eoq_conv_fused_us"] + t["fwd_bn_passes_us"], t["fwd_conv_with_sum_dump_us"] + t["fwd_bn_passes_us"]]
        t["fwd_slowdown_with_bn"] = [x / t["fwd_eoq_conv_fused_us"] for x in t["fwd_bn_total_us"]]
        t["bwd_slowdown_with_bn"] = t["bwd_bn_passes_and_Qe_us"] / t["bwd_eoq_error_head_us"]
        t["layer"] = f"{l.name} {l.h}x{l.w} {l.c_in}->{l.c_out} k{l.k} batch {l.n}"
        rows.append(t)
    assert eoq.eoq_last_status(h) & ~eoq.EOQ_DEV_SQ_ZERO == 0
    eoq.eoq_destroy(h)
    print(json.dumps({"probe": "bn_vs_fixup", "unit": "us per call (graph replay)", "layers": rows}), flush=True)


# ----------------------------------------------------------------------------------------------- launcher

def launch_ranks(args, argv):
    """--gpus N without a launcher environment: start N ranks of this script (torch.distributed.run, one node,
    rendezvous on 127.0.0.1) and pass their output through; rank 0 prints the JSON line."""
    import socket

    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + argv
    return subprocess.call(cmd)


def run_dry(args):
    """--dry-run: the rank plumbing alone (rendezvous, barrier, max-over-ranks of a stand-in timing, one JSON line
    from rank 0) on CPU with gloo; what the multi-rank tests drive."""
    from paper_2105_13890_b200 import ranks

    world, rank, _ = ranks.world()
    ranks.init("gloo")
    ranks.barrier(sync_cuda=False)
    ms = ranks.max_over_ranks([10.0 + rank], device="cpu")[0]
    ranks.barrier(sync_cuda=False)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "n_gpus": world, "dry_run": True, "ms_per_step": ms / args.steps,
                          "value": ranks.whole_job_rate(1e12, args.steps, ms, world) / 1e12, "unit": "TOPS",
                          "scaling": "weak", "config": {"parallelism": f"replicas x{world}"}}), flush=True)
    ranks.finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="eoq", choices=["eoq", "reference"])
    ap.add_argument("--workload", default="resnet18")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--ref-batch", type=int, default=0,
                    help="batch of the CPU-oracle step timed beside the GPU run (0 = the workload's own batch)")
    ap.add_argument("--ref-arm-batch", type=int, default=1, help="batch of each step of --impl reference")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--eager", action="store_true", help="launch call by call on one stream instead of replaying a CUDA graph")
    ap.add_argument("--independent", action="store_true", help="time the layer units on independent synthetic tensors (no glue)")
    ap.add_argument("--stochastic", action="store_true", help="stochastic rounding in the update (an extension; default: nearest even)")
    ap.add_argument("--probe", default=None, choices=["mma_i8", "bn_vs_fixup"],
                    help="mma_i8: measure the INT8 tensor-pipe figures; bn_vs_fixup: batch normalisation against the fused Fixup epilogue")
    ap.add_argument("--probe-seconds", type=float, default=2.0, help="length of each sustained probe loop")
    ap.add_argument("--int8-peaks", default=None, help="JSON printed by --probe, to report fractions of those figures too")
    ap.add_argument("--step-only", action="store_true",
                    help="run the warm-up and timed steps and nothing else (launch lists under a profiler)")
    ap.add_argument("--dry-run", action="store_true", help="rank plumbing only, on CPU with gloo (tests)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_ranks(args, sys.argv[1:]))
    if args.dry_run:
        run_dry(args)
    elif args.probe == "bn_vs_fixup":
        run_bn_compare(args)
    elif args.probe:
        run_probe(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()

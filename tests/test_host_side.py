"""CPU-only checks of the product's host side: the library loads and exports the header's symbols, argument
validation that needs no device, workload op counts, and the two-rank timing reduction over gloo."""
import os
import re
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import oracle
from paper_2105_13890_b200 import build, eoq, ranks, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    build.build_lib()
    header = open(os.path.join(ROOT, "include", "eoq.h")).read()
    declared = set(re.findall(r"EOQ_API[^;(]*?\b(eoq_\w+)\s*\(", header))
    assert {"eoq_conv_fwd", "eoq_conv_dgrad", "eoq_conv_wgrad", "eoq_quantize", "eoq_update"} <= declared
    lib = eoq.lib()
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(eoq.EXPORTS)


def test_workspace_size_and_argument_checks_need_no_device():
    d = eoq.conv_desc(64, 56, 56, 64, 64, 3, 3, 1, 1)
    assert eoq.eoq_workspace_size(d, eoq.EOQ_PASS_DGRAD) >= 64 * 56 * 56 * 64 * 4 + 64 * 9 * 64
    assert eoq.eoq_workspace_size(d, eoq.EOQ_PASS_WGRAD) >= 64 * 9 * 64 * 8
    assert eoq.eoq_workspace_size(d, eoq.EOQ_PASS_FWD) % 256 == 0
    with pytest.raises(eoq.EoqError) as e:
        eoq.eoq_workspace_size(eoq.conv_desc(1, 8, 8, 12, 16, 3, 3, 1, 1), 0)
    assert e.value.status == eoq.EOQ_ERR_ALIGNMENT
    with pytest.raises(eoq.EoqError) as e:
        eoq.eoq_workspace_size(eoq.conv_desc(1, 2, 2, 16, 16, 7, 7, 1, 0), 0)
    assert e.value.status == eoq.EOQ_ERR_BAD_ARG
    with pytest.raises(eoq.EoqError) as e:
        eoq.eoq_workspace_size(eoq.conv_desc(1, 32, 32, 16, 16, 9, 9, 1, 4), 0)
    assert e.value.status == eoq.EOQ_ERR_UNSUPPORTED
    assert "alignment" in eoq.status_string(eoq.EOQ_ERR_ALIGNMENT)


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a device")
def test_create_fails_loudly_without_a_gpu():
    with pytest.raises(eoq.EoqError):
        eoq.eoq_create(0)


def test_workload_op_counts_and_fixup_coefficient():
    r18, r20, r50 = workloads.resnet18(), workloads.resnet20(), workloads.resnet50()
    # algorithmic work per step: 3 passes per conv, 2 for the first layer, true channel counts
    assert r18.total_macs == pytest.approx(340.65e9, rel=1e-4) and len(r18.layers) == 20
    assert r20.total_macs == pytest.approx(15.6e9, rel=2e-3) and len(r20.layers) == 21
    assert r50.total_macs == pytest.approx(388.6e9, rel=1e-3) and len(r50.layers) == 53
    assert sum(l.weight_elems for l in r18.layers) == pytest.approx(11.2e6, rel=2e-3)
    # the paper's other two networks (Sec. 5.1, 5.4): 3.66 and 0.253 GMAC per image forward
    r34, r110 = workloads.resnet34(), workloads.resnet110()
    assert len(r34.layers) == 36 and r34.L == 16 and len(r110.layers) == 111 and r110.L == 54
    assert sum(l.macs for l in r34.layers) / r34.batch == pytest.approx(3.663e9, rel=1e-3)
    assert sum(l.macs for l in r110.layers) / r110.batch == pytest.approx(0.2531e9, rel=1e-3)
    assert workloads.get("resnet110", 4).batch == 4 and workloads.get("resnet34", 2).layers[0].k == 7
    for L, m in ((8, 2), (9, 2), (16, 3), (54, 2)):
        assert workloads.fixup_alpha(L, m) == pytest.approx(oracle.fixup_alpha(L, m), rel=1e-15)
    layer = r18.layers[1]
    z = np.random.default_rng(0).standard_normal((layer.c_out, 3, 3, layer.c_in))
    assert np.array_equal(workloads.init_weight_f32(layer, r18, z), oracle.fixup_weights_f32(z, 9 * 64, 8, 2))
    stem = workloads.init_weight_f32(r18.layers[0], r18, np.ones((64, 7, 7, 16)))
    assert not stem[..., 3:].any() and stem[0, 0, 0, 0] == np.float32(np.sqrt(2.0 / 147))


def _rank_main(rank, port, out):
    os.environ.update(WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    ranks.init("gloo")
    ranks.barrier(sync_cuda=False)
    ms = ranks.max_over_ranks([10.0 + 5.0 * rank, 7.0 - rank])
    rate = ranks.whole_job_rate(100.0, 4, ms[0], ranks.world()[0])
    out.put((rank, ms, rate))
    ranks.finish()


def test_two_rank_timing_reduction_over_gloo():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, rate in got:
        assert ms == [15.0, 7.0]                       # the slowest rank's time on every rank
        assert rate == pytest.approx(2 * 100.0 * 4 / 0.015)


# ------------------------------------------------------------------ data-parallel replicas: the exchange that keeps them exact

def _sq_with_global_max(a, p_a, m_global):
    """SQ of a local share under the maximum of the whole batch: a sentinel carrying that maximum joins the share."""
    codes, p, _ = oracle.sq_int(np.concatenate([np.asarray(a, dtype=np.int64).reshape(-1), [m_global]]), p_a)
    return codes[:-1].reshape(np.shape(a)), p


def _replica_main(rank, port, out):
    """One of two replicas holding half of the batch: local oracle partials, all-reduced as the library's hook
    all-reduces them (maxima of the scale quantizers, sums of the gradients)."""
    import torch.distributed as dist
    from oracle import ConvDesc
    from paper_2105_13890_b200 import synth

    os.environ.update(WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    ranks.init("gloo")

    def allmax(v):
        t = torch.tensor([int(v)], dtype=torch.int64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return int(t.item())

    def allsum(a):
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.int64))
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return t.numpy()

    full = ConvDesc(4, 8, 8, 16, 32, 3, 3, 1, 1)
    d = ConvDesc(2, 8, 8, 16, 32, 3, 3, 1, 1)
    sl = slice(2 * rank, 2 * rank + 2)
    x0 = synth.relu_codes((full.n, full.h, full.w, full.c_in), 71, 0)[sl]
    w = synth.int8_uniform((full.c_out, 3, 3, full.c_in), 71, 1, -20, 20)
    e0 = synth.normal_codes((full.n, full.ho, full.wo, full.c_out), 71, 2)[sl]
    b1, gamma, b2, p0 = -2, 118, 3, -12
    fwd = oracle.layer_forward(d, x0, b1, w, gamma, b2)                      # per sample: no exchange
    e1 = e0.astype(np.int64) * fwd["mask"]
    m1 = allmax(np.abs(gamma * e1).max())                                       # max behind e3 = Q_e(gamma e1)
    e3, p3 = _sq_with_global_max(gamma * e1, p0 - 7, m1)
    s_e1 = int(allsum(np.array([e1.sum()]))[0])
    B = oracle.conv_dgrad_acc(d, e3.astype(np.int8), w)
    e4, p4 = _sq_with_global_max(B, p3 - 7, allmax(np.abs(B).max()))            # max behind e4 = Q_e(e3 * w)
    G = allsum(oracle.conv_wgrad_acc(d, e3.astype(np.int8), x0, b1))            # exact integer sums in front of Q_g
    g, pg, _ = oracle.sq_int(G, p3 - 7)
    out.put((rank, e3, p3, e4, p4, g, pg, s_e1))
    ranks.finish()


def test_two_replicas_exchange_maxima_and_integer_sums_and_match_one_device():
    from oracle import ConvDesc
    from paper_2105_13890_b200 import synth

    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_replica_main, args=(r, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the whole batch in one process
    full = ConvDesc(4, 8, 8, 16, 32, 3, 3, 1, 1)
    x0 = synth.relu_codes((full.n, full.h, full.w, full.c_in), 71, 0)
    w = synth.int8_uniform((full.c_out, 3, 3, full.c_in), 71, 1, -20, 20)
    e0 = synth.normal_codes((full.n, full.ho, full.wo, full.c_out), 71, 2)
    fwd = oracle.layer_forward(full, x0, -2, w, 118, 3)
    ref = oracle.layer_backward(full, e0, -12, fwd["mask"], fwd["x2"], x0, -2, w, 118)
    e3 = np.concatenate([got[0][1], got[1][1]])
    e4 = np.concatenate([got[0][3], got[1][3]])
    assert np.array_equal(e3, ref["e3"]) and got[0][2] == got[1][2] == ref["p3"]
    assert np.array_equal(e4, ref["e4"]) and got[0][4] == got[1][4] == ref["p4"]
    for r in (0, 1):                                                            # every replica holds the same gradient
        assert np.array_equal(got[r][5], ref["g_w"]) and got[r][6] == ref["p_gw"] and got[r][7] == ref["sum_e1"]


def test_bench_launcher_starts_the_ranks_itself():
    """`bench.py --gpus 2` without a launcher environment starts two ranks (here on CPU with gloo, plumbing only) and
    rank 0 prints one JSON line for the whole job."""
    import json
    import subprocess
    import sys

    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--steps", "4"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["config"]["parallelism"] == "replicas x2"
    assert line["ms_per_step"] == pytest.approx(11.0 / 4)                       # the slower rank's 11 ms over 4 steps

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

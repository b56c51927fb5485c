"""The N > 1 path of bench.py without GPUs: the method does not shard across GPUs, so N ranks are N
independent replicas; what the ranks share is the timing reduction (max over ranks) and the rule that
only rank 0 reports.  Run here as two `gloo` ranks on CPU."""
import json
import os
import subprocess
import sys

import pytest
import torch.multiprocessing as mp

from helpers import ROOT


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 2.0 + rank                       # rank 1 is the slow replica
    worst = bench.max_over_ranks(local_ms, world, "cpu")
    rate = bench.whole_job_rate(world, 100, 64 << 20, worst * 1e-3)
    dist.barrier()
    out.put((rank, worst, rate))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    world, port = 2, _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, worst, rate in got:
        assert worst == 3.0                                   # the slow replica's time, on every rank
        assert rate == pytest.approx(2 * 100 * (64 << 20) / 3.0e-3 / 1e9)


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25, 1, "cpu") == 1.25
    assert bench.whole_job_rate(1, 8, 1 << 20, 1e-3) == pytest.approx(8 * (1 << 20) / 1e-3 / 1e9)


def test_reference_arm_under_torchrun_only_rank0_reports():
    """`bench.py --impl reference` launched as two ranks: rank 0 times the CPU oracle and prints the
    one JSON line, the other rank exits 0 without work."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--workload", "cfg3",
           "--steps", "1", "--warmup", "0"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["unit"] == "GB/s"
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["value"] == rec["value"]
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["e2e"]["d2h_bytes_per_step"] == 0
    assert rec["gpu_launches"] == 0

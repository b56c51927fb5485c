"""One process per GPU on the one GPU at hand: `bench.py --sharded --same-device` as two and three
processes that all use cuda:0.  Each owns its share of the rank buffers, reads the others' through
CUDA IPC mappings and runs the phases with a (gloo) barrier after each; bench.py itself compares
every rank buffer with the root's message before it prints.  The processes' kernels never wait for
one another: every kernel runs to its end on its own."""
import json
import os
import subprocess
import sys

import pytest

from helpers import ROOT

pytestmark = pytest.mark.gpu


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("world,workload", [(2, "P12x262149r5"), (3, "P64x4194317r17")])
def test_processes_sharing_one_device(world, workload):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(world),
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "bench.py"), "--sharded", "--same-device", "--gpus", str(world), "--workload", workload,
           "--steps", "3", "--warmup", "1"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, (res.stdout[-1500:], res.stderr[-3000:])
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == world and rec["scaling"] == "strong" and rec["value"] > 0
    assert rec["config"]["phases"] >= 2 and rec["config"]["nvlink_bytes_per_step"] > 0
    assert rec["native"]["nvlink_bytes_per_step"] >= rec["config"]["nvlink_bytes_per_step"]  # tuned never sends more over the links

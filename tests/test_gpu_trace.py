"""What the executors did, counted on the device, against the oracle.

Final buffers equal the root's message under any schedule that reaches every rank, so buffer parity
alone cannot tell an executor that performs all the native ring's redundant messages from one
that skips them.  bcast_exec_traced makes the kernels add, per message of the plan, the bytes they
store for it; here those device-side counts must equal the oracle's `len` message by message, and
their per-rank sums the oracle's per-process byte counters (Sections III-A and IV count exactly
these: 56 vs 44 ring messages for P = 8).  Also: the bounded wait of the bulk-copy kernel."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from helpers import ROOT
from paper_1603_06809_b200 import bcast as B
from paper_1603_06809_b200 import workloads as W
from gpu_harness import RankBuffers

pytestmark = pytest.mark.gpu

TRACE_MODES = [B.BCAST_EXEC_WALK, B.BCAST_EXEC_WALK_PLAN_ORDER, B.BCAST_EXEC_WALK_BULK, B.BCAST_EXEC_STEPS]
TRACE_IDS = ["walk", "walk_plan_order", "walk_bulk", "steps"]
VARIANTS = [B.BCAST_NATIVE, B.BCAST_TUNED, B.BCAST_DOUBLING]
VARIANT_IDS = ["native", "tuned", "doubling"]

SHAPES = [W.Workload("trace_p8", 8, 0, 1 << 20, 11), W.Workload("trace_p12_odd", 12, 5, 256 * 1024 + 5, 12),
          W.Workload("trace_p16_cut", 16, 15, 16 * (65536 + 2051), 13), W.Workload("trace_p33_tiny", 33, 32, 700, 14),
          W.Workload("trace_p64_odd", 64, 17, (4 << 20) + 13, 15), W.Workload("trace_p255_empty", 255, 254, 12 * 1024, 16)]


def traced_counts(wl, variant, mode):
    msg = W.message_bytes(wl.seed, wl.nbytes)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, variant)
    counts = torch.zeros(max(1, B.bcast_plan_num_xfers(plan)), dtype=torch.int64, device="cuda:0")
    B.bcast_exec_traced(bufs.pointers(), plan, torch.cuda.current_stream(), mode, counts)
    torch.cuda.synchronize()
    B.bcast_exec_status(plan)
    assert bufs.all_equal_message() and bufs.guards_intact()
    return plan, counts.cpu().numpy()[: B.bcast_plan_num_xfers(plan)]


@pytest.mark.parametrize("mode", TRACE_MODES, ids=TRACE_IDS)
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
@pytest.mark.parametrize("wl", SHAPES, ids=lambda w: w.name)
def test_every_message_is_performed_in_full_exactly_once(oracle, wl, variant, mode):
    if variant == B.BCAST_DOUBLING and wl.P & (wl.P - 1):
        pytest.skip("recursive doubling needs a power of two")
    plan, counts = traced_counts(wl, variant, mode)
    ref = oracle.simulate(wl.P, wl.root, wl.nbytes, variant)
    assert len(counts) == len(ref.schedule)
    assert np.array_equal(counts, ref.col("len"))                       # bytes per message
    for ph in (0, 1):                                                  # per process and phase
        sel = ref.col("phase") == ph
        sent = np.bincount(ref.col("src")[sel], weights=counts[sel], minlength=wl.P).astype(np.uint64)
        recv = np.bincount(ref.col("dst")[sel], weights=counts[sel], minlength=wl.P).astype(np.uint64)
        assert np.array_equal(sent, ref.bytes_sent[ph])
        assert np.array_equal(recv, ref.bytes_recv[ph])


def test_native_moves_more_than_tuned_on_the_device(oracle):
    wl = W.CFG3
    _, native = traced_counts(wl, B.BCAST_NATIVE, B.BCAST_EXEC_WALK)
    _, tuned = traced_counts(wl, B.BCAST_TUNED, B.BCAST_EXEC_WALK)
    assert len(native) == 63 + 64 * 63 and len(tuned) == 63 + 3840       # 4032 vs 3840 ring messages
    assert int(tuned.sum()) == 63 * wl.nbytes                            # every non-root byte written once
    assert int(native.sum()) > int(tuned.sum())


def test_traced_refuses_graph_mode_and_null_counters():
    wl = W.Workload("trace_bad", 4, 0, 4096, 2)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, W.message_bytes(wl.seed, wl.nbytes))
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    counts = torch.zeros(16, dtype=torch.int64, device="cuda:0")
    with pytest.raises(B.BcastError) as e:
        B.bcast_exec_traced(bufs.pointers(), plan, None, B.BCAST_EXEC_GRAPH, counts)
    assert e.value.code == B.BCAST_ERR_INVAL
    with pytest.raises(B.BcastError) as e:
        B.bcast_exec_traced(bufs.pointers(), plan, None, B.BCAST_EXEC_WALK, 0)
    assert e.value.code == B.BCAST_ERR_INVAL


BOUNDED_WAIT_CHILD = r"""
import sys
import torch
sys.path.insert(0, sys.argv[1])
sys.path.insert(0, sys.argv[1] + "/tests")
from paper_1603_06809_b200 import bcast as B, workloads as W
from gpu_harness import RankBuffers
wl = W.Workload("wait", 12, 5, 12 * 65536, 3)
msg = W.message_bytes(wl.seed, wl.nbytes)
bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_NATIVE)
B.bcast_exec_mode(bufs.pointers(), plan, None, B.BCAST_EXEC_WALK_BULK)
torch.cuda.synchronize()
assert bufs.all_equal_message() and bufs.guards_intact()       # the kernel ran to its normal end
try:
    B.bcast_exec_status(plan)
    print("STATUS ok")
except B.BcastError as e:
    print("STATUS", e.code)
B.bcast_exec_status(plan)                                       # the flag was cleared by the read
print("SECOND ok")
"""


def test_bounded_wait_reports_timeout_and_the_kernel_still_completes():
    """With a poll budget of zero every wait of the bulk-copy kernel runs out at once: each worker
    raises the flag and then waits on under its second bound, so the copies all land, the result is
    complete, bcast_exec_status reports BCAST_ERR_TIMEOUT once and BCAST_OK afterwards.  Nothing
    here can hang or fault: the copies are ordinary, only the budget is small.  (A child process,
    because the budget is read from the environment when a plan is first executed.)"""
    for limit, want in (("0", f"STATUS {B.BCAST_ERR_TIMEOUT}"), ("", "STATUS ok")):
        env = dict(os.environ)
        env.pop("BCAST_BULK_SPIN_LIMIT", None)
        if limit:
            env["BCAST_BULK_SPIN_LIMIT"] = limit
        out = subprocess.run([sys.executable, "-c", BOUNDED_WAIT_CHILD, ROOT], env=env, capture_output=True, text=True,
                             timeout=300)
        assert out.returncode == 0, out.stderr[-2000:]
        assert want in out.stdout and "SECOND ok" in out.stdout, out.stdout

"""bcast_exec_static: the broadcast for callers that cannot allocate device memory.

Some users of this library run inside programs that gave all device memory to their own pool at
start-up, or that work under a fixed memory budget, or that cannot afford the device-wide stall of
cudaMalloc: for them the library offers an entry point whose kernel tables live in a fixed array
inside the library itself.  This file checks, through the C ABI, that it delivers exactly what the
allocating entry point bcast_exec() delivers, on two calls in a row that share the array, and that a
plan too large for the array is refused.  It is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

from paper_1603_06809_b200 import bcast as B
from paper_1603_06809_b200 import workloads as W
from gpu_harness import RankBuffers

pytestmark = pytest.mark.gpu


def run(entry, wl, variant, msg):
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, variant)
    entry(bufs.pointers(), plan, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert bufs.guards_intact()
    return bufs.to_host()


def test_static_matches_allocating_entry_point_twice_in_a_row():
    # two different plans back to back: the second call finds the first call's tables in the array
    cases = [(W.Workload("static_a", 12, 5, 256 * W.KiB + 5, 41), B.BCAST_TUNED),
             (W.Workload("static_b", 33, 32, 4 * W.MiB + 3, 42), B.BCAST_NATIVE),
             (W.Workload("static_a", 12, 5, 256 * W.KiB + 5, 41), B.BCAST_TUNED)]
    for wl, variant in cases:
        msg = W.message_bytes(wl.seed, wl.nbytes)
        got = run(B.bcast_exec_static, wl, variant, msg)
        want = run(B.bcast_exec, wl, variant, msg)
        assert np.array_equal(got, want)                 # byte work: bit-exact
        assert (got == msg[None, :]).all()


def test_static_same_plan_twice_without_reset_between():
    wl = W.CFG3
    msg = W.message_bytes(wl.seed, wl.nbytes)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    st = torch.cuda.current_stream()
    B.bcast_exec_static(bufs.pointers(), plan, st)
    B.bcast_exec_static(bufs.pointers(), plan, st)       # same stream: ordered after the first
    torch.cuda.synchronize()
    assert bufs.all_equal_message() and bufs.guards_intact()
    ref = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
    B.bcast_exec(ref.pointers(), plan, st)
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(bufs.view, ref.view))


def test_static_refuses_host_memory():
    wl = W.Workload("static_bad", 4, 0, 4096, 2)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, W.message_bytes(wl.seed, wl.nbytes))
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    good = bufs.pointers()
    host = torch.zeros(8192, dtype=torch.uint8).pin_memory()
    with pytest.raises(B.BcastError) as e:
        B.bcast_exec_static([good[0], host.data_ptr(), good[2], good[3]], plan, torch.cuda.current_stream())
    assert e.value.code == B.BCAST_ERR_INVAL
    B.bcast_exec_static(good, plan, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert bufs.all_equal_message() and bufs.guards_intact()


def test_static_refuses_plans_beyond_its_capacity():
    P, n = 1024, 64 * 1024
    plan = B.bcast_plan(P, 0, n, B.BCAST_NATIVE)        # about 4 * P * P bytes of hop lists: too large
    dev = torch.zeros((P, n), dtype=torch.uint8, device="cuda:0")
    with pytest.raises(B.BcastError) as e:
        B.bcast_exec_static([dev[k].data_ptr() for k in range(P)], plan, torch.cuda.current_stream())
    assert e.value.code == B.BCAST_ERR_CAPACITY
    torch.cuda.synchronize()
    assert not dev.any()                                  # nothing was launched
    assert "scratch" in B.bcast_strerror(B.BCAST_ERR_CAPACITY)


def test_static_allocates_no_device_memory():
    # the property the entry point exists for: on a plan that bcast_exec never saw (so no cached
    # device tables can stand in), the driver's count of free device memory must not move
    wl = W.Workload("static_noalloc", 24, 3, 3 * W.MiB + 7, 43)
    msg = W.message_bytes(wl.seed, wl.nbytes)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
    st = torch.cuda.current_stream()
    warm = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_NATIVE)       # module and kernel loading happen here
    B.bcast_exec_static(bufs.pointers(), warm, st)
    torch.cuda.synchronize()
    bufs.reset()
    fresh = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    B.bcast_exec_static(bufs.pointers(), fresh, st)
    B.bcast_exec_static(bufs.pointers(), fresh, st)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    B.bcast_exec_status(fresh)                                         # no device state was created for this plan
    assert bufs.all_equal_message() and bufs.guards_intact()


def test_static_refuses_a_capturing_stream():
    # its copy into the shared array must not be recorded into a graph: the call says so instead
    wl = W.Workload("static_capture", 8, 0, 65536, 44)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, W.message_bytes(wl.seed, wl.nbytes))
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    B.bcast_exec_static(bufs.pointers(), plan, torch.cuda.current_stream())   # first call on the device: outside capture
    torch.cuda.synchronize()
    bufs.reset()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    code = None
    with torch.cuda.graph(graph, stream=side):
        try:
            B.bcast_exec_static(bufs.pointers(), plan, side)
        except B.BcastError as e:
            code = e.code
    assert code == B.BCAST_ERR_INVAL
    torch.cuda.synchronize()
    B.bcast_exec_static(bufs.pointers(), plan, torch.cuda.current_stream())   # still usable afterwards
    torch.cuda.synchronize()
    assert bufs.all_equal_message() and bufs.guards_intact()


def test_static_falls_back_when_the_boundary_lists_do_not_fit():
    # P = 512 with an odd scatter size: hop lists (4 P^2 bytes) fit into the built-in array, the merged
    # boundary lists on top of them do not; the call then walks cut segments in two parts instead
    wl = W.Workload("static_p512", 512, 77, 512 * 2051 + 9, 45)
    msg = W.message_bytes(wl.seed, wl.nbytes)
    got = run(B.bcast_exec_static, wl, B.BCAST_TUNED, msg)
    assert (got == msg[None, :]).all()
    want = run(B.bcast_exec, wl, B.BCAST_TUNED, msg)
    assert np.array_equal(got, want)

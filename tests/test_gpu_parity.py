"""GPU parity: the CUDA executors, called through the C ABI, against the CPU oracle.

Byte work, so the bar is bit-exact: every rank buffer equals the oracle's buffer of that rank
element by element, guard zones around the buffers are untouched, and the plan that was executed
equals the oracle's schedule and counters (tests/test_plan_parity.py checks the latter on CPU)."""
import ctypes

import numpy as np
import pytest
import torch

from paper_1603_06809_b200 import bcast as B
from paper_1603_06809_b200 import workloads as W
from gpu_harness import RankBuffers, run_broadcast

pytestmark = pytest.mark.gpu

MODES = [B.BCAST_EXEC_WALK, B.BCAST_EXEC_STEPS, B.BCAST_EXEC_GRAPH, B.BCAST_EXEC_WALK_PLAN_ORDER,
         B.BCAST_EXEC_WALK_BULK, B.BCAST_EXEC_AUTO]
MODE_IDS = ["walk", "steps", "graph", "walk_plan_order", "walk_bulk", "auto"]
VARIANTS = [B.BCAST_NATIVE, B.BCAST_TUNED]
VARIANT_IDS = ["native", "tuned"]


def check_against_oracle(oracle, wl, variant, mode, shift=0, repeats=1):
    msg = W.message_bytes(wl.seed, wl.nbytes)
    plan, bufs = run_broadcast(wl.P, wl.root, wl.nbytes, variant, mode, msg, shift=shift, repeats=repeats)
    B.bcast_exec_status(plan)                       # no bounded wait ran out
    ref = oracle.simulate(wl.P, wl.root, wl.nbytes, variant, message=msg)
    got = bufs.to_host()
    assert got.shape == ref.bufs.shape
    assert np.array_equal(got, ref.bufs)
    assert bufs.guards_intact()
    x = B.bcast_plan_xfers(plan)
    assert len(x) == len(ref.schedule)
    assert np.array_equal(x["len"].astype(np.int64), ref.col("len"))
    assert np.array_equal(x["src_rank"].astype(np.int64), ref.col("src"))
    assert np.array_equal(x["dst_rank"].astype(np.int64), ref.col("dst"))
    assert np.array_equal(x["offset"].astype(np.int64), ref.col("offset"))
    for ph in (0, 1):
        assert np.array_equal(B.bcast_plan_bytes_recv(plan, ph), ref.bytes_recv[ph])
        assert np.array_equal(B.bcast_plan_bytes_sent(plan, ph), ref.bytes_sent[ph])


# ---- configurations 1-3 in full, element by element, all executors
@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
@pytest.mark.parametrize("wl", [W.CFG1, W.CFG2, W.CFG3], ids=lambda w: w.name)
def test_configs_1_to_3(oracle, wl, variant, mode):
    check_against_oracle(oracle, wl, variant, mode)


# ---- configuration 2 with every root
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
def test_cfg2_all_roots(oracle, variant):
    for wl in W.cfg2_all_roots():
        check_against_oracle(oracle, wl, variant, B.BCAST_EXEC_WALK)
    check_against_oracle(oracle, W.cfg2_all_roots()[7], variant, B.BCAST_EXEC_STEPS)


# ---- small, ragged and degenerate shapes: several tiles plus ragged tails, chunks shorter than a
# word, empty chunks, nbytes < P, nbytes = 0, P = 1, P = 2
SMALL = [(1, 0, 1000), (2, 1, 1), (2, 0, 4097), (3, 1, 2), (5, 3, 4), (7, 6, 12288), (9, 4, 524287),
         (10, 0, 40), (16, 15, 65521), (17, 5, 1048576), (33, 32, 100003), (255, 254, 12288),
         (256, 255, 12288), (13, 2, 13 * 16 * 256 * 4 + 5), (6, 2, 0), (64, 63, 63), (129, 77, 2560000)]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
@pytest.mark.parametrize("P,root,n", SMALL)
def test_small_and_ragged(oracle, P, root, n, variant, mode):
    check_against_oracle(oracle, W.Workload(f"P{P}_{n}", P, root, n, 7000 + P), variant, mode)


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_buffers_at_odd_16_byte_offsets(oracle, mode):
    """Rank buffers only need 16-byte alignment, not more."""
    for shift in (16, 48, 240):
        check_against_oracle(oracle, W.Workload("shifted", 12, 5, 100001, 99), B.BCAST_TUNED, mode, shift=shift)


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_repeated_execution_and_new_buffers(oracle, mode):
    """A plan can be executed again (work counters return to zero) and with other buffers."""
    wl = W.Workload("again", 24, 23, 4 * W.MiB + 3, 123)
    check_against_oracle(oracle, wl, B.BCAST_TUNED, mode, repeats=3)
    msg = W.message_bytes(wl.seed, wl.nbytes)
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_NATIVE)
    for rep in range(2):
        bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg, shift=16 * rep)
        B.bcast_exec_mode(bufs.pointers(), plan, torch.cuda.current_stream(), mode)
        torch.cuda.synchronize()
        assert bufs.all_equal_message() and bufs.guards_intact()


def test_runs_on_a_side_stream(oracle):
    wl = W.Workload("side", 12, 3, 3 * W.MiB + 1, 5)
    msg = W.message_bytes(wl.seed, wl.nbytes)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    for mode in MODES:
        bufs.reset()
        torch.cuda.synchronize()
        B.bcast_exec_mode(bufs.pointers(), plan, side, mode)
        side.synchronize()
        assert bufs.all_equal_message() and bufs.guards_intact()


# ---- configuration 4 at full size, in the launch configuration the benchmark times (WALK): every
# rank buffer compared with the root's message on the device, sampled ranks against the oracle's
# buffers on the host, schedule and counters against the oracle
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
def test_cfg4_full_size(oracle, variant):
    wl = W.CFG4
    msg = W.message_bytes(wl.seed, wl.nbytes)
    for mode in (B.BCAST_EXEC_WALK_BULK, B.BCAST_EXEC_AUTO):    # AUTO (what bench.py times) is the register walk at this size
        plan, bufs = run_broadcast(wl.P, wl.root, wl.nbytes, variant, mode, msg)
        assert bufs.all_equal_message() and bufs.guards_intact()
        B.bcast_exec_status(plan)
        if mode == B.BCAST_EXEC_WALK_BULK:
            del bufs
            torch.cuda.empty_cache()
    ref = oracle.simulate(wl.P, wl.root, wl.nbytes, variant, message=msg)
    for k in (0, 1, 37, 62, 63, 64, 99):
        assert np.array_equal(bufs.view[k].cpu().numpy(), ref.bufs[k])
    x = B.bcast_plan_xfers(plan)
    assert np.array_equal(x["len"].astype(np.int64), ref.col("len"))
    assert B.bcast_plan_total_bytes(plan) == int(ref.col("len").sum())


def test_cfg4_steps_executor():
    wl = W.CFG4
    msg = W.message_bytes(wl.seed, wl.nbytes)
    _, bufs = run_broadcast(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED, B.BCAST_EXEC_GRAPH, msg)
    assert bufs.all_equal_message() and bufs.guards_intact()


# ---- configuration 5: the sweep.  Points the oracle finishes in seconds are compared element by
# element on the host; the large ones (up to 34 GB of rank buffers) rank by rank against the
# message on the device, which is what the oracle's buffers equal (MPI broadcast semantics).
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
def test_sweep(oracle, variant):
    for wl in W.sweep():
        if wl.total_bytes <= 600 * W.MiB:
            check_against_oracle(oracle, wl, variant, B.BCAST_EXEC_WALK)
        else:
            msg = W.message_bytes(wl.seed, wl.nbytes)
            plan, bufs = run_broadcast(wl.P, wl.root, wl.nbytes, variant, B.BCAST_EXEC_AUTO, msg)
            assert bufs.all_equal_message() and bufs.guards_intact(), wl.name
            B.bcast_exec_status(plan)
            ref = oracle.simulate(wl.P, wl.root, wl.nbytes, variant)          # schedule and counters only
            assert B.bcast_plan_total_bytes(plan) == int(ref.col("len").sum())
            del bufs
            torch.cuda.empty_cache()


def test_sweep_steps_executor_medium_points(oracle):
    for wl in W.sweep():
        if wl.total_bytes <= 128 * W.MiB:
            check_against_oracle(oracle, wl, B.BCAST_TUNED, B.BCAST_EXEC_STEPS)


# ---- the paper's own experiment shapes (Section V): every point element by element, both variants
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
def test_paper_experiment_shapes(oracle, variant):
    for wl in W.paper_experiments():
        if wl.total_bytes <= 300 * W.MiB:
            check_against_oracle(oracle, wl, variant, B.BCAST_EXEC_WALK)
        else:
            msg = W.message_bytes(wl.seed, wl.nbytes)
            plan, bufs = run_broadcast(wl.P, wl.root, wl.nbytes, variant, B.BCAST_EXEC_WALK, msg)
            assert bufs.all_equal_message() and bufs.guards_intact(), wl.name
            ref = oracle.simulate(wl.P, wl.root, wl.nbytes, variant)
            assert B.bcast_plan_total_bytes(plan) == int(ref.col("len").sum())
            del bufs
            torch.cuda.empty_cache()


# ---- scatter + recursive-doubling allgather (power-of-two P), every executor
DOUBLING_CASES = [W.CFG1, W.CFG3, W.Workload("P2", 2, 1, 4097, 21), W.Workload("P4", 4, 3, 3, 22),
                  W.Workload("P16_odd", 16, 5, 1_000_003, 23), W.Workload("P32", 32, 0, 12288, 24),
                  W.Workload("P256", 256, 255, 4 * W.MiB + 1, 25), W.Workload("P128_empty", 128, 9, 100, 26)]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("wl", DOUBLING_CASES, ids=lambda w: w.name)
def test_recursive_doubling_variant(oracle, wl, mode):
    check_against_oracle(oracle, wl, B.BCAST_DOUBLING, mode)


# ---- the largest accepted rank count (the P > 128 kernel instantiation with an 8 KiB pointer argument)
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
def test_largest_rank_count(oracle, variant):
    wl = W.Workload("P1024", B.BCAST_MAX_RANKS, 1000, 300_007, 77)
    for mode in (B.BCAST_EXEC_WALK, B.BCAST_EXEC_WALK_PLAN_ORDER, B.BCAST_EXEC_STEPS):
        check_against_oracle(oracle, wl, variant, mode)


# ---- offsets beyond 4 GiB: 64-bit arithmetic in the planner, the slice list and the kernels
def test_message_larger_than_4_gib(oracle):
    P, root, n = 3, 2, (4 << 30) + 4097
    msg = torch.empty(n, dtype=torch.uint8, device="cuda:0")
    g = torch.Generator(device="cuda:0").manual_seed(5)
    msg.random_(0, 256, generator=g)
    bufs = [torch.full((n + 512,), 0xC3, dtype=torch.uint8, device="cuda:0") for _ in range(P)]
    views = [b[256:256 + n] for b in bufs]
    views[root].copy_(msg)
    for mode in (B.BCAST_EXEC_WALK, B.BCAST_EXEC_STEPS, B.BCAST_EXEC_WALK_BULK):
        for k in range(P):
            if k != root:
                views[k].fill_(W.poison_byte(k))
        plan = B.bcast_plan(P, root, n, B.BCAST_TUNED)
        B.bcast_exec_mode([v.data_ptr() for v in views], plan, torch.cuda.current_stream(), mode)
        torch.cuda.synchronize()
        for k in range(P):
            assert torch.equal(views[k], msg)
            assert bool((bufs[k][:256] == 0xC3).all()) and bool((bufs[k][256 + n:] == 0xC3).all())
        ref = oracle.simulate(P, root, n, B.BCAST_TUNED)                 # schedule only
        x = B.bcast_plan_xfers(plan)
        assert np.array_equal(x["offset"].astype(np.int64), ref.col("offset"))
        assert np.array_equal(x["len"].astype(np.int64), ref.col("len"))
    del bufs, views, msg
    torch.cuda.empty_cache()


# ---- one plan, two sets of rank buffers, two streams at the same time
def test_same_plan_on_two_streams_with_different_buffers(oracle):
    wl = W.Workload("two_streams", 24, 7, 8 * W.MiB + 5, 91)
    msg_a = W.message_bytes(wl.seed, wl.nbytes)
    msg_b = W.message_bytes(wl.seed + 1, wl.nbytes)
    a = RankBuffers(wl.P, wl.root, wl.nbytes, msg_a)
    b = RankBuffers(wl.P, wl.root, wl.nbytes, msg_b)
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    B.bcast_exec(a.pointers(), plan, torch.cuda.current_stream())     # first execution builds the tables
    torch.cuda.synchronize()
    a.reset()
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    for _ in range(3):
        B.bcast_exec(a.pointers(), plan, s1)
        B.bcast_exec(b.pointers(), plan, s2)
    torch.cuda.synchronize()
    assert a.all_equal_message() and b.all_equal_message()
    assert a.guards_intact() and b.guards_intact()
    ref = oracle.simulate(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED, message=msg_b)
    assert np.array_equal(b.to_host(), ref.bufs)


# ---- host-memory entry point
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
def test_exec_host(oracle, variant):
    wl = W.Workload("host", 12, 5, 1 * W.MiB + 77, 31)
    msg = W.message_bytes(wl.seed, wl.nbytes)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, np.zeros(wl.nbytes, np.uint8))   # root NOT pre-filled
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, variant)
    host_msg = torch.from_numpy(msg.copy()).pin_memory()
    outs = torch.zeros((wl.P, wl.nbytes), dtype=torch.uint8).pin_memory()
    out_list = [outs[k] for k in range(wl.P)]
    out_list[3] = None
    B.bcast_exec_host(bufs.pointers(), plan, torch.cuda.current_stream(), B.BCAST_EXEC_WALK, host_msg, out_list)
    ref = oracle.simulate(wl.P, wl.root, wl.nbytes, variant, message=msg)
    got = outs.numpy()
    for k in range(wl.P):
        if k == 3:
            assert not got[k].any()
        else:
            assert np.array_equal(got[k], ref.bufs[k])
    assert bufs.guards_intact()


def test_exec_host_argument_errors():
    wl = W.Workload("host_bad", 4, 1, 4096, 3)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, W.message_bytes(wl.seed, wl.nbytes))
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    ptrs = (ctypes.c_void_p * 4)(*bufs.pointers())
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert B._lib.bcast_exec_host(ptrs, plan.handle, st, B.BCAST_EXEC_WALK, None, None) == B.BCAST_ERR_INVAL
    assert B._lib.bcast_exec_host(None, plan.handle, st, B.BCAST_EXEC_WALK, None, None) == B.BCAST_ERR_INVAL
    host = torch.from_numpy(W.message_bytes(9, wl.nbytes)).pin_memory()
    assert B._lib.bcast_exec_host(ptrs, plan.handle, st, 99, ctypes.c_void_p(host.data_ptr()), None) == B.BCAST_ERR_INVAL
    # an empty message needs no host pointer
    empty = B.bcast_plan(4, 1, 0, B.BCAST_TUNED)
    assert B._lib.bcast_exec_host(ptrs, empty.handle, st, B.BCAST_EXEC_WALK, None, None) == B.BCAST_OK


# ---- argument errors are refused before anything is launched
def test_exec_rejects_bad_buffers():
    wl = W.Workload("bad", 4, 0, 4096, 1)
    msg = W.message_bytes(wl.seed, wl.nbytes)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    good = bufs.pointers()
    host_pinned = torch.zeros(8192, dtype=torch.uint8).pin_memory()
    host_plain = np.zeros(8192, dtype=np.uint8)
    for bad in ([good[0], 0, good[2], good[3]],                  # NULL
                [good[0], good[1] + 8, good[2], good[3]],        # misaligned
                [good[0], good[1], good[1], good[3]],            # duplicate
                [good[0], good[0] + 1024, good[2], good[3]],     # overlapping
                [good[0], host_pinned.data_ptr(), good[2], good[3]],          # pinned host memory
                [good[0], host_plain.ctypes.data // 16 * 16 + 16, good[2], good[3]]):   # pageable host memory
        with pytest.raises(B.BcastError) as e:
            B.bcast_exec(bad, plan)
        assert e.value.code == B.BCAST_ERR_INVAL
    torch.cuda.synchronize()
    assert not bufs.all_equal_message()          # nothing ran
    B.bcast_exec(good, plan)
    torch.cuda.synchronize()
    assert bufs.all_equal_message() and bufs.guards_intact()


# ---- the node-aware broadcast (Section II) through every executor, and its bytes counted on the device
SMP_WORKLOADS = [(W.Workload("smp_p12", 12, 5, 256 * 1024 + 5, 51), 4), (W.Workload("smp_p24", 24, 13, 24 * 40961, 52), 6),
                 (W.Workload("smp_p129", 129, 0, 524287, 53), 24), (W.Workload("smp_p100", 100, 63, (8 << 20) + 1, 54), 8),
                 (W.Workload("smp_one_node", 9, 2, 70001, 55), 16), (W.Workload("smp_tiny", 33, 20, 700, 56), 8)]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
@pytest.mark.parametrize("wl,c", SMP_WORKLOADS, ids=lambda x: x.name if hasattr(x, "name") else f"c{x}")
def test_node_aware_broadcast(oracle, wl, c, variant, mode):
    msg = W.message_bytes(wl.seed, wl.nbytes)
    plan, bufs = run_broadcast(wl.P, wl.root, wl.nbytes, variant, mode, msg, ranks_per_node=c)
    B.bcast_exec_status(plan)
    ref = oracle.simulate(wl.P, wl.root, wl.nbytes, variant, message=msg, ranks_per_node=c)
    assert np.array_equal(bufs.to_host(), ref.bufs)
    assert bufs.guards_intact()
    x = B.bcast_plan_xfers(plan)
    assert np.array_equal(x["len"].astype(np.int64), ref.col("len"))
    assert np.array_equal(x["dep"], ref.col("dep"))
    if mode in (B.BCAST_EXEC_WALK, B.BCAST_EXEC_WALK_BULK, B.BCAST_EXEC_STEPS):
        bufs.reset()
        counts = torch.zeros(len(x), dtype=torch.int64, device="cuda:0")
        B.bcast_exec_traced(bufs.pointers(), plan, torch.cuda.current_stream(), mode, counts)
        torch.cuda.synchronize()
        assert np.array_equal(counts.cpu().numpy(), ref.col("len"))       # every message performed in full, once
        assert bufs.all_equal_message()


# ---- seeded random shapes: every kind of slice (whole, cut by one boundary, cut by several, message
# tail), every variant, the executors in turn
def _random_cases(count, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(count):
        P = int(rng.choice([2, 3, 5, 9, 17, 31, 48, 64, 100, 129, 200, 255, 300]))
        kind = i % 4
        if kind == 0:
            n = int(rng.integers(1, 4 * P))                      # chunks of a few bytes, some empty
        elif kind == 1:
            n = int(rng.integers(P * 40, P * 700))               # several boundaries per 512-byte segment
        elif kind == 2:
            n = int(rng.integers(P * 3000, P * 9000))            # one boundary per segment at most
        else:
            n = int(rng.integers(1 << 20, 3 << 20))              # a megabyte or so, odd
        cases.append((P, int(rng.integers(0, P)), n, int(rng.integers(0, 3)), i))
    return cases


@pytest.mark.parametrize("P,root,n,variant,i", _random_cases(48, 20261130))
def test_random_shapes(oracle, P, root, n, variant, i):
    if variant == B.BCAST_DOUBLING and P & (P - 1):
        variant = B.BCAST_TUNED
    mode = MODES[i % len(MODES)]
    check_against_oracle(oracle, W.Workload(f"random_{i}", P, root, n, 900 + i), variant, mode, shift=16 * (i % 2))
    # and the same shape node-aware, or spread over a partition, with the bytes counted on the device
    msg = W.message_bytes(900 + i, n)
    if variant != B.BCAST_DOUBLING and i % 3 == 0:
        c = int(1 + (i * 7) % max(1, P // 2))
        plan, bufs = run_broadcast(P, root, n, variant, mode, msg, ranks_per_node=c)
        ref = oracle.simulate(P, root, n, variant, message=msg, ranks_per_node=c)
        assert np.array_equal(bufs.to_host(), ref.bufs) and bufs.guards_intact()
    if i % 3 == 1:
        G = int(min(P, 2 + i % 5))
        bufs = RankBuffers(P, root, n, msg)
        plan = B.bcast_plan(P, root, n, variant)
        shard = B.bcast_shard_create(plan, G)
        counts = torch.zeros(max(1, B.bcast_plan_num_xfers(plan)), dtype=torch.int64, device="cuda:0")
        st = torch.cuda.current_stream()
        torch.cuda.synchronize()
        B.bcast_shard_exec(shard, bufs.pointers(), [0] * G, [st] * G, counts)
        torch.cuda.synchronize()
        ref = oracle.simulate(P, root, n, variant, message=msg)
        assert np.array_equal(bufs.to_host(), ref.bufs) and bufs.guards_intact()
        assert np.array_equal(counts.cpu().numpy()[: len(ref.schedule)], ref.col("len"))

"""Host-side checks without a GPU: the library loads and exports every symbol of include/bcast.h,
and the planner's schedule, dependency indices and per-rank counters equal the oracle's
bit for bit (the planner uses the closed form of the binomial tree, the oracle runs the
per-process loops of the paper's listing: two derivations of the same schedule)."""
import ctypes
import os
import re

import numpy as np
import pytest

from helpers import ROOT
from paper_1603_06809_b200 import bcast as B
from paper_1603_06809_b200 import workloads as W

FIELDS = ("phase", "step", "src_rank", "dst_rank", "chunk", "nchunks", "offset", "len", "dep")


def plan_matrix(plan):
    x = B.bcast_plan_xfers(plan)
    return np.stack([x[f].astype(np.int64) for f in FIELDS], axis=1) if len(x) else np.zeros((0, 9), np.int64)


def assert_plan_equals_oracle(oracle, P, root, n, variant):
    plan = B.bcast_plan(P, root, n, variant)
    ref = oracle.simulate(P, root, n, variant)
    mine = plan_matrix(plan)
    assert mine.shape == ref.schedule.shape
    assert (mine == ref.schedule).all()
    assert B.bcast_plan_scatter_size(plan) == ref.scatter_size
    assert B.bcast_plan_total_bytes(plan) == int(ref.col("len").sum())
    for ph in (B.BCAST_PHASE_SCATTER, B.BCAST_PHASE_RING):
        assert (B.bcast_plan_bytes_sent(plan, ph) == ref.bytes_sent[ph]).all()
        assert (B.bcast_plan_bytes_recv(plan, ph) == ref.bytes_recv[ph]).all()
        assert (B.bcast_plan_msgs_sent(plan, ph) == ref.msgs_sent[ph]).all()
        assert (B.bcast_plan_msgs_recv(plan, ph) == ref.msgs_recv[ph]).all()
    # CSR over steps: L + P - 1 steps, each holding the messages with that (phase, step)
    sb = B.bcast_plan_step_begin(plan)
    L = (P - 1).bit_length()
    nsteps = (2 * L if variant == B.BCAST_DOUBLING else L + P - 1) if P > 1 else 0
    assert B.bcast_plan_num_steps(plan) == nsteps and len(sb) == nsteps + 1
    assert sb[0] == 0 and sb[-1] == len(mine) and (np.diff(sb) >= 0).all()
    for s in range(nsteps):
        rows = mine[sb[s]:sb[s + 1]]
        want = (0, s) if s < L else (1, s - L)
        assert ((rows[:, 0] == want[0]) & (rows[:, 1] == want[1])).all()
    B.bcast_plan_free(plan)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "bcast.h")).read()
    declared = set(re.findall(r"\b(bcast_[a-z_]+)\s*\(", header))
    assert declared == set(B.SYMBOLS)
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_1603_06809_b200", "libbcast_b200.so"))
    for name in declared:
        assert hasattr(lib, name), name


def test_binding_constants_match_header():
    header = open(os.path.join(ROOT, "include", "bcast.h")).read()
    pairs = dict(re.findall(r"\b(BCAST_[A-Z_]+)\s*=\s*(-?\d+)", header))
    assert len(pairs) == 19
    for name, value in pairs.items():
        assert getattr(B, name) == int(value), name
    assert B.BCAST_MAX_RANKS == int(re.search(r"#define BCAST_MAX_RANKS (\d+)", header).group(1))
    assert B.BCAST_STATIC_SCRATCH_BYTES == 2 << 20 and "#define BCAST_STATIC_SCRATCH_BYTES (2u << 20)" in header


def test_xfer_layout_matches_header():
    assert B.XFER_DTYPE.itemsize == 48
    assert [B.XFER_DTYPE.fields[f][1] for f in FIELDS] == [0, 4, 8, 12, 16, 20, 24, 32, 40]


@pytest.mark.parametrize("variant", [B.BCAST_NATIVE, B.BCAST_TUNED])
def test_plan_equals_oracle_small_grid(oracle, variant):
    for P in list(range(1, 34)) + [63, 64, 65]:
        for root in sorted({0, P // 3, P - 1}):
            for n in (0, 1, P - 1, P, P + 1, 97, 12288, 1000003):
                assert_plan_equals_oracle(oracle, P, root, n, variant)


@pytest.mark.parametrize("variant", [B.BCAST_NATIVE, B.BCAST_TUNED])
@pytest.mark.parametrize("wl", [W.CFG1, W.CFG2, W.CFG3, W.CFG4], ids=lambda w: w.name)
def test_plan_equals_oracle_configs(oracle, wl, variant):
    assert_plan_equals_oracle(oracle, wl.P, wl.root, wl.nbytes, variant)


@pytest.mark.parametrize("variant", [B.BCAST_NATIVE, B.BCAST_TUNED])
def test_plan_equals_oracle_all_roots_cfg2(oracle, variant):
    for wl in W.cfg2_all_roots():
        assert_plan_equals_oracle(oracle, wl.P, wl.root, wl.nbytes, variant)


@pytest.mark.parametrize("variant", [B.BCAST_NATIVE, B.BCAST_TUNED])
def test_plan_equals_oracle_sweep(oracle, variant):
    sweep = W.sweep()
    assert len(sweep) == 45
    for wl in sweep:
        assert_plan_equals_oracle(oracle, wl.P, wl.root, wl.nbytes, variant)


@pytest.mark.parametrize("variant", [B.BCAST_NATIVE, B.BCAST_TUNED])
def test_plan_equals_oracle_paper_experiment_shapes(oracle, variant):
    shapes = W.paper_experiments()
    assert len(shapes) == 3 * 7 + 5 * 3 + 6
    for wl in shapes:
        assert_plan_equals_oracle(oracle, wl.P, wl.root, wl.nbytes, variant)


def test_plan_equals_oracle_doubling(oracle):
    """Scatter + recursive-doubling allgather (power-of-two P): schedule, `dep` and counters."""
    for P in (1, 2, 4, 8, 16, 32, 64, 128, 256, 1024):
        for root in sorted({0, P // 3, P - 1}):
            for n in (0, 1, P - 1, P, P + 1, 12288, 1000003):
                assert_plan_equals_oracle(oracle, P, root, n, B.BCAST_DOUBLING)
    for wl in (W.CFG1, W.CFG3):
        assert_plan_equals_oracle(oracle, wl.P, wl.root, wl.nbytes, B.BCAST_DOUBLING)
    for P in (3, 12, 100, 255):
        with pytest.raises(B.BcastError) as e:
            B.bcast_plan(P, 0, 1000, B.BCAST_DOUBLING)
        assert e.value.code == B.BCAST_ERR_INVAL


def test_plan_largest_rank_count(oracle):
    assert_plan_equals_oracle(oracle, B.BCAST_MAX_RANKS, 1000, 5_000_011, B.BCAST_TUNED)


def test_plan_argument_errors():
    for args in [(0, 0, 10, 1), (-1, 0, 10, 1), (B.BCAST_MAX_RANKS + 1, 0, 10, 1), (4, 4, 10, 1), (4, -1, 10, 1),
                 (4, 0, 10, 3), (4, 0, 10, -1), (4, 0, 2**64 - 1, 1)]:
        with pytest.raises(B.BcastError) as e:
            B.bcast_plan(*args)
        assert e.value.code == B.BCAST_ERR_INVAL
    # out == NULL
    assert B._lib.bcast_plan(4, 0, 10, 1, None) == B.BCAST_ERR_INVAL
    # NULL plan: accessors answer 0 / NULL, free is a no-op
    assert B._lib.bcast_plan_num_xfers(None) == 0 and not B._lib.bcast_plan_xfers(None)
    assert not B._lib.bcast_plan_bytes_sent(None, 0)
    B._lib.bcast_plan_free(None)
    plan = B.bcast_plan(4, 0, 10, 1)
    assert not B._lib.bcast_plan_bytes_sent(plan.handle, 4) and not B._lib.bcast_plan_bytes_sent(plan.handle, -1)
    assert not B.bcast_plan_bytes_sent(plan, B.BCAST_PHASE_NODE_LAST).any()     # phases of the node-aware broadcast: unused here
    assert B.bcast_strerror(B.BCAST_ERR_INVAL) == "invalid argument" and B.bcast_strerror(0) == "success"


def test_exec_argument_errors_need_no_gpu():
    plan = B.bcast_plan(4, 0, 64, 1)
    assert B._lib.bcast_exec(None, plan.handle, None) == B.BCAST_ERR_INVAL
    assert B._lib.bcast_exec((ctypes.c_void_p * 4)(16, 32, 48, 64), None, None) == B.BCAST_ERR_INVAL
    assert B._lib.bcast_exec_mode((ctypes.c_void_p * 4)(16, 32, 48, 64), plan.handle, None, 7) == B.BCAST_ERR_INVAL
    assert B.bcast_exec_num_launches(plan, B.BCAST_EXEC_WALK) == 1
    assert B.bcast_exec_num_launches(plan, B.BCAST_EXEC_WALK_PLAN_ORDER) == 1
    assert B.bcast_exec_num_launches(plan, B.BCAST_EXEC_WALK_BULK) == 1
    assert B.bcast_exec_num_launches(plan, B.BCAST_EXEC_AUTO) == 1
    B.bcast_exec_status(plan)                                  # never executed: nothing to report
    assert B._lib.bcast_exec_status(None) == B.BCAST_ERR_INVAL
    assert B.bcast_exec_num_launches(plan, B.BCAST_EXEC_STEPS) == 2 + 3
    assert B.bcast_exec_num_launches(B.bcast_plan(1, 0, 64, 1), B.BCAST_EXEC_WALK) == 0
    assert B.bcast_exec_num_launches(B.bcast_plan(4, 0, 0, 1), B.BCAST_EXEC_STEPS) == 0
    # P = 255, 12 KiB: the last four chunks are empty, but every step still moves something
    assert B.bcast_exec_num_launches(B.bcast_plan(255, 254, 12288, 0), B.BCAST_EXEC_STEPS) == 8 + 254


def test_exec_without_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    plan = B.bcast_plan(4, 0, 64, 1)
    with pytest.raises(B.BcastError) as e:
        B.bcast_exec([4096, 8192, 12288, 16384], plan)
    assert e.value.code == B.BCAST_ERR_CUDA


@pytest.mark.parametrize("variant", [B.BCAST_NATIVE, B.BCAST_TUNED, B.BCAST_DOUBLING])
def test_walk_order_respects_every_dependency(oracle, variant):
    """The order in which the one-launch executor performs the messages of a chunk (both of its
    modes): the same messages as the oracle's schedule has for that chunk, each once; a message
    never before the message named by its `dep`; replayed in that order, the sender always holds
    the chunk already and in the end every rank holds it."""
    for P, root, n in [(2, 1, 64), (8, 0, 1 << 12), (10, 3, 12345), (12, 5, 256 << 10), (33, 32, 100003),
                       (64, 17, (16 << 20) + 13), (100, 63, 64 << 20), (255, 254, 12288)]:
        if variant == B.BCAST_DOUBLING and P & (P - 1):
            continue
        plan = B.bcast_plan(P, root, n, variant)
        ref = oracle.simulate(P, root, n, variant)
        S = ref.scatter_size
        sched = ref.schedule
        for c in sorted({0, 1, P // 2, P - 2, P - 1} & set(range(P))):
            clen = min((c + 1) * S, n) - min(c * S, n)
            want = [i for i in range(len(sched))
                    if sched[i, 7] > 0 and sched[i, 4] <= c < sched[i, 4] + sched[i, 5] and clen > 0]
            plan_order = B.bcast_plan_walk_order(plan, c, B.BCAST_EXEC_WALK_PLAN_ORDER)
            walk_order = B.bcast_plan_walk_order(plan, c, B.BCAST_EXEC_WALK)
            assert list(plan_order) == want
            assert sorted(walk_order) == want
            if variant == B.BCAST_NATIVE:
                assert list(walk_order) == want          # ranks are re-written: plan order is kept
            for order in (plan_order, walk_order):
                pos = {int(m): k for k, m in enumerate(order)}
                holders = {root}
                for m in order:
                    dep = int(sched[m, 8])
                    if variant != B.BCAST_DOUBLING:
                        assert dep < 0 or dep in pos       # the producer covers this chunk too
                    if dep in pos:                         # (doubling: `dep` is about the block's first chunk)
                        assert pos[dep] < pos[int(m)]
                    assert int(sched[m, 2]) in holders
                    holders.add(int(sched[m, 3]))
                if want:
                    assert holders == set(range(P))
    with pytest.raises(B.BcastError):
        B.bcast_plan_walk_order(B.bcast_plan(4, 0, 64, 1), 4)
    with pytest.raises(B.BcastError):
        B.bcast_plan_walk_order(B.bcast_plan(4, 0, 64, 1), 0, B.BCAST_EXEC_STEPS)


def test_walk_order_reads_follow_writes_closely():
    """Tuned ring: in the one-launch executor's order a copy is read at most a few messages after
    it was written (one level of the dependency tree), never ~P messages later as in plan order."""
    P, root, n = 100, 63, 64 << 20
    plan = B.bcast_plan(P, root, n, B.BCAST_TUNED)
    x = B.bcast_plan_xfers(plan)
    L = (P - 1).bit_length()
    worst_walk, worst_plan = 0, 0
    for c in range(P):
        for mode in (B.BCAST_EXEC_WALK, B.BCAST_EXEC_WALK_PLAN_ORDER):
            order = B.bcast_plan_walk_order(plan, c, mode)
            written_at = {}
            worst = 0
            for k, m in enumerate(order):
                src, dst = int(x[m]["src_rank"]), int(x[m]["dst_rank"])
                if src in written_at:
                    worst = max(worst, k - written_at[src])
                written_at[dst] = k
            if mode == B.BCAST_EXEC_WALK:
                worst_walk = max(worst_walk, worst)
            else:
                worst_plan = max(worst_plan, worst)
    assert worst_walk <= 2 * (L + 1)
    assert worst_plan > P // 2


def test_plan_equals_oracle_random_shapes(oracle):
    """Randomly drawn (P, root, nbytes, variant): planner and oracle agree on everything."""
    from hypothesis import given, settings, strategies as st

    @settings(max_examples=150, deadline=None, derandomize=True)
    @given(st.integers(1, 200), st.data())
    def check(P, data):
        root = data.draw(st.integers(0, P - 1))
        n = data.draw(st.one_of(st.integers(0, 4 * P + 3), st.integers(0, 1 << 22)))
        variants = [B.BCAST_NATIVE, B.BCAST_TUNED] + ([B.BCAST_DOUBLING] if P & (P - 1) == 0 else [])
        assert_plan_equals_oracle(oracle, P, root, n, data.draw(st.sampled_from(variants)))
    check()


# ---- the node-aware broadcast (Section II): planner (closed form per group) == oracle (simulation)
SMP_SHAPES = [(12, 5, 1000, 4), (12, 0, 4096, 3), (10, 7, 777, 3), (24, 13, 24 * 100 + 1, 6), (9, 2, 64, 4), (16, 15, 5000, 4),
              (7, 3, 50, 2), (33, 20, 33 * 31, 8), (6, 5, 3, 5), (100, 63, 1 << 20, 8), (129, 0, 524287, 24), (64, 17, (1 << 20) + 13, 64),
              (8, 3, 100, 1), (5, 4, 0, 2), (1, 0, 10, 4)]


@pytest.mark.parametrize("variant", [B.BCAST_NATIVE, B.BCAST_TUNED], ids=["native", "tuned"])
@pytest.mark.parametrize("P,root,n,c", SMP_SHAPES)
def test_node_aware_plan_equals_oracle(oracle, P, root, n, c, variant):
    plan = B.bcast_plan_smp(P, root, n, variant, c)
    ref = oracle.simulate(P, root, n, variant, ranks_per_node=c)
    mine = plan_matrix(plan)
    assert mine.shape == ref.schedule.shape
    assert (mine == ref.schedule).all()                       # every field, `dep` included
    assert B.bcast_plan_scatter_size(plan) == ref.scatter_size
    assert B.bcast_plan_ranks_per_node(plan) == c and B.bcast_plan_num_chunks(plan) == -(-P // c)
    for ph in range(4):
        assert (B.bcast_plan_bytes_sent(plan, ph) == ref.bytes_sent[ph]).all()
        assert (B.bcast_plan_bytes_recv(plan, ph) == ref.bytes_recv[ph]).all()
        assert (B.bcast_plan_msgs_sent(plan, ph) == ref.msgs_sent[ph]).all()
        assert (B.bcast_plan_msgs_recv(plan, ph) == ref.msgs_recv[ph]).all()
    # CSR over steps: every step holds the messages of one (phase, step)
    sb = B.bcast_plan_step_begin(plan)
    assert sb[0] == 0 and sb[-1] == len(mine) and (np.diff(sb) >= 0).all()
    seen = []
    for s in range(len(sb) - 1):
        rows = mine[sb[s]:sb[s + 1]]
        if len(rows):
            assert len({(int(r[0]), int(r[1])) for r in rows}) == 1
            seen.append((int(rows[0, 0]), int(rows[0, 1])))
    assert seen == sorted(set(seen), key=lambda ps: ({2: 0, 0: 1, 1: 2, 3: 3}[ps[0]], ps[1]))
    # the hop order of the walk respects every dependency here too
    x = B.bcast_plan_xfers(plan)
    for chunk in range(B.bcast_plan_num_chunks(plan)):
        for mode in (B.BCAST_EXEC_WALK, B.BCAST_EXEC_WALK_PLAN_ORDER):
            order = B.bcast_plan_walk_order(plan, chunk, mode)
            pos = {int(m): i for i, m in enumerate(order)}
            for m in order:
                d = int(x["dep"][m])
                if d >= 0 and d in pos:
                    assert pos[d] < pos[int(m)]


def test_node_aware_plan_argument_errors():
    for args in [(8, 0, 100, B.BCAST_TUNED, 0), (8, 0, 100, B.BCAST_DOUBLING, 2), (8, 9, 100, B.BCAST_TUNED, 2), (0, 0, 1, 0, 1)]:
        with pytest.raises(B.BcastError):
            B.bcast_plan_smp(*args)

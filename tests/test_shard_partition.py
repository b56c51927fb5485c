"""The ranks of a plan spread over G GPUs, host side (no GPU): every hop lands in exactly one
(phase, GPU) kernel; replaying the kernels phase by phase -- a GPU reading other GPUs' buffers only
as they were when the phase began -- leaves the oracle's buffers; what crosses a GPU boundary is what
the oracle's schedule says crosses it."""
import numpy as np
import pytest

from paper_1603_06809_b200 import bcast as B
from paper_1603_06809_b200 import workloads as W

VARIANTS = [(B.BCAST_NATIVE, "native"), (B.BCAST_TUNED, "tuned"), (B.BCAST_DOUBLING, "doubling")]
SHAPES = [(8, 0, 8 * 64 + 3, 2), (8, 3, 1000, 4), (10, 7, 10 * 33, 3), (12, 5, 4096 + 5, 4), (16, 15, 16 * 100, 8),
          (33, 32, 33 * 17 + 2, 4), (64, 17, 64 * 50 + 13, 8), (7, 2, 5, 2), (6, 1, 6000, 6), (9, 0, 900, 1)]


def chunk_range(plan, c):
    n, S = B.bcast_plan_nbytes(plan), B.bcast_plan_scatter_size(plan)
    return min(c * S, n), min((c + 1) * S, n)


def replay_by_phases(plan, shard, msg, root):
    """Perform the partition's hop lists on host buffers, phase by phase.  Reads of a buffer owned by
    another GPU see the state at the start of the phase; reads of an own buffer see live data."""
    P, n = B.bcast_plan_num_ranks(plan), B.bcast_plan_nbytes(plan)
    G, nph = B.bcast_shard_num_gpus(shard), B.bcast_shard_num_phases(shard)
    x = B.bcast_plan_xfers(plan)
    owner = B.bcast_shard_rank_gpu(shard)
    bufs = np.zeros((P, n), dtype=np.uint8)
    for k in range(P):
        bufs[k, :] = W.poison_byte(k)
    bufs[root, :] = msg
    done = np.zeros(len(x), dtype=np.int64)          # bytes performed per message
    for ph in range(nph):
        before = bufs.copy()
        for g in range(G):
            for c in range(P):
                lo, hi = chunk_range(plan, c)
                for m in B.bcast_shard_hops(shard, ph, g, c):
                    s, d = int(x["src_rank"][m]), int(x["dst_rank"][m])
                    assert owner[d] == g and x["chunk"][m] <= c < x["chunk"][m] + x["nchunks"][m]
                    src = bufs if owner[s] == g else before
                    bufs[d, lo:hi] = src[s, lo:hi]
                    done[m] += hi - lo
    return bufs, done


@pytest.mark.parametrize("variant,vname", VARIANTS, ids=[v[1] for v in VARIANTS])
@pytest.mark.parametrize("P,root,n,G", SHAPES)
def test_phase_replay_equals_the_oracle(oracle, variant, vname, P, root, n, G):
    if variant == B.BCAST_DOUBLING and P & (P - 1):
        pytest.skip("recursive doubling needs a power of two")
    plan = B.bcast_plan(P, root, n, variant)
    shard = B.bcast_shard_create(plan, G)
    msg = W.message_bytes(5 + P, n)
    ref = oracle.simulate(P, root, n, variant, message=msg)
    bufs, done = replay_by_phases(plan, shard, msg, root)
    assert np.array_equal(bufs, ref.bufs)                               # nothing was read before it had arrived
    assert np.array_equal(done, ref.col("len"))                         # every hop in exactly one kernel
    # what crosses a GPU boundary, from the oracle's schedule and the same rank-to-GPU map
    owner = B.bcast_shard_rank_gpu(shard)
    assert np.array_equal(owner, np.arange(P) * G // P)
    cross = owner[ref.col("src")] != owner[ref.col("dst")]
    assert B.bcast_shard_crossing_bytes(shard) == int(ref.col("len")[cross].sum())
    assert B.bcast_shard_crossing_msgs(shard) == int(cross.sum())
    assert np.array_equal(B.bcast_shard_msg_gpu(shard), owner[ref.col("dst")])
    first, last = B.bcast_shard_msg_phase(shard), B.bcast_shard_msg_phase(shard, last=True)
    moving = ref.col("len") > 0
    assert (first[moving] >= 0).all() and (last >= first).all() and (first[~moving] == -1).all()
    if G == 1:
        assert B.bcast_shard_num_phases(shard) == (1 if n and P > 1 else 0) and B.bcast_shard_crossing_bytes(shard) == 0


def test_tuned_saves_on_the_links_what_it_saves_in_total():
    # contiguous groups: in the ring every chunk crosses each of the G group boundaries once, except
    # where the receiver already holds it (tuned); the scatter crosses at most log2 levels
    P, G, n = 64, 8, 64 * 4096
    cross = {}
    for variant in (B.BCAST_NATIVE, B.BCAST_TUNED):
        plan = B.bcast_plan(P, 0, n, variant)
        shard = B.bcast_shard_create(plan, G)
        cross[variant] = B.bcast_shard_crossing_bytes(shard)
        assert B.bcast_shard_num_phases(shard) <= G + 7
    assert cross[B.BCAST_TUNED] < cross[B.BCAST_NATIVE]
    assert cross[B.BCAST_TUNED] <= G * n                                  # about (G / P) (P - 1) n ...
    assert cross[B.BCAST_TUNED] >= (G - 1) * n - n                        # ... and not much less


def test_custom_rank_map_and_argument_errors():
    plan = B.bcast_plan(6, 0, 600, B.BCAST_TUNED)
    shard = B.bcast_shard_create(plan, 2, [0, 1, 0, 1, 0, 1])             # interleaved: every ring hop crosses
    x = B.bcast_plan_xfers(plan)
    ring = x["phase"] == B.BCAST_PHASE_RING
    assert B.bcast_shard_crossing_msgs(shard) >= int(ring.sum())
    for bad in ([0, 1, 2, 0, 0, 0], [0, 0, 0]):
        with pytest.raises(B.BcastError):
            B.bcast_shard_create(plan, 2, bad)
    for g in (0, 7):
        with pytest.raises(B.BcastError):
            B.bcast_shard_create(plan, g)
    with pytest.raises(B.BcastError):
        B.bcast_shard_hops(shard, 99, 0, 0)

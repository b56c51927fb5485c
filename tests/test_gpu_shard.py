"""The partitioned executor on the one GPU at hand: G = 2, 4, 8 "GPUs" of the partition all mapped to
device 0, each with a stream of its own (the same code path as on G devices; the peer pointers happen
to be local).  Buffers against the oracle bit for bit, and the bytes counted per message on the device
against the oracle's schedule."""
import numpy as np
import pytest
import torch

from paper_1603_06809_b200 import bcast as B
from paper_1603_06809_b200 import workloads as W
from gpu_harness import RankBuffers

pytestmark = pytest.mark.gpu

VARIANTS = [B.BCAST_NATIVE, B.BCAST_TUNED, B.BCAST_DOUBLING]
VARIANT_IDS = ["native", "tuned", "doubling"]
SHAPES = [W.Workload("shard_p8", 8, 0, 1 << 20, 21), W.Workload("shard_p12_odd", 12, 5, 256 * 1024 + 5, 22),
          W.Workload("shard_p64_odd", 64, 17, (4 << 20) + 13, 23), W.Workload("shard_p33_tiny", 33, 32, 700, 24),
          W.Workload("shard_p100", 100, 63, 100 * 40961, 25), W.Workload("shard_p16", 16, 9, 16 * 70000, 26)]


def run_sharded(oracle, wl, variant, G, per_phase=False, rank_gpu=None):
    msg = W.message_bytes(wl.seed, wl.nbytes)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, variant)
    shard = B.bcast_shard_create(plan, G, rank_gpu)
    counts = torch.zeros(max(1, B.bcast_plan_num_xfers(plan)), dtype=torch.int64, device="cuda:0")
    torch.cuda.synchronize()
    if per_phase:
        # what one process per GPU does, phase by phase with a barrier in between: here one process
        # plays all of them in turn
        st = torch.cuda.current_stream()
        for ph in range(B.bcast_shard_num_phases(shard)):
            for g in range(G):
                B.bcast_shard_exec_phase(shard, bufs.pointers(), ph, g, st, counts)
            torch.cuda.synchronize()
    else:
        streams = [torch.cuda.Stream() for _ in range(G)]
        for rep in range(2):                                    # the second run must wait for the first on every stream
            if rep:
                torch.cuda.synchronize()
                bufs.reset()
                counts.zero_()
                torch.cuda.synchronize()
            B.bcast_shard_exec(shard, bufs.pointers(), [0] * G, streams, counts)
        torch.cuda.synchronize()
    ref = oracle.simulate(wl.P, wl.root, wl.nbytes, variant, message=msg)
    assert np.array_equal(bufs.to_host(), ref.bufs)
    assert bufs.guards_intact()
    assert np.array_equal(counts.cpu().numpy()[: len(ref.schedule)], ref.col("len"))
    return shard


@pytest.mark.parametrize("G", [2, 4, 8])
@pytest.mark.parametrize("variant", VARIANTS, ids=VARIANT_IDS)
@pytest.mark.parametrize("wl", SHAPES, ids=lambda w: w.name)
def test_partitions_on_one_device_match_the_oracle(oracle, wl, variant, G):
    if variant == B.BCAST_DOUBLING and wl.P & (wl.P - 1):
        pytest.skip("recursive doubling needs a power of two")
    run_sharded(oracle, wl, variant, G)


@pytest.mark.parametrize("variant", VARIANTS[:2], ids=VARIANT_IDS[:2])
def test_phase_by_phase_entry_point(oracle, variant):
    run_sharded(oracle, W.Workload("shard_phase", 24, 7, 24 * 5000 + 1, 27), variant, 3, per_phase=True)


def test_interleaved_rank_map(oracle):
    P = 10
    run_sharded(oracle, W.Workload("shard_interleaved", P, 4, 10 * 3000 + 7, 28), B.BCAST_TUNED, 2,
                rank_gpu=[r % 2 for r in range(P)])


def test_shard_exec_rejects_misplaced_and_bad_arguments():
    wl = W.Workload("shard_bad", 4, 0, 4096, 2)
    bufs = RankBuffers(wl.P, wl.root, wl.nbytes, W.message_bytes(wl.seed, wl.nbytes))
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, B.BCAST_TUNED)
    shard = B.bcast_shard_create(plan, 2)
    st = torch.cuda.current_stream()
    host = torch.zeros(8192, dtype=torch.uint8).pin_memory()
    good = bufs.pointers()
    with pytest.raises(B.BcastError) as e:
        B.bcast_shard_exec(shard, [good[0], host.data_ptr(), good[2], good[3]], [0, 0], [st, st])
    assert e.value.code == B.BCAST_ERR_INVAL
    with pytest.raises(B.BcastError) as e:
        B.bcast_shard_exec(shard, good, [0, 99], [st, st])             # rank buffers are not on device 99
    assert e.value.code == B.BCAST_ERR_INVAL
    with pytest.raises(B.BcastError) as e:
        B.bcast_shard_exec_phase(shard, good, 99, 0, st)
    assert e.value.code == B.BCAST_ERR_INVAL
    B.bcast_shard_exec(shard, good, [0, 0], [st, st])
    torch.cuda.synchronize()
    assert bufs.all_equal_message() and bufs.guards_intact()


def test_node_aware_plan_over_partitions(oracle):
    # nodes of the plan and GPUs of the partition are independent groupings of the ranks
    wl = W.Workload("shard_smp", 24, 13, 24 * 40961, 29)
    msg = W.message_bytes(wl.seed, wl.nbytes)
    for variant in (B.BCAST_NATIVE, B.BCAST_TUNED):
        bufs = RankBuffers(wl.P, wl.root, wl.nbytes, msg)
        plan = B.bcast_plan_smp(wl.P, wl.root, wl.nbytes, variant, 6)
        shard = B.bcast_shard_create(plan, 4)
        counts = torch.zeros(B.bcast_plan_num_xfers(plan), dtype=torch.int64, device="cuda:0")
        streams = [torch.cuda.Stream() for _ in range(4)]
        torch.cuda.synchronize()
        B.bcast_shard_exec(shard, bufs.pointers(), [0] * 4, streams, counts)
        torch.cuda.synchronize()
        ref = oracle.simulate(wl.P, wl.root, wl.nbytes, variant, message=msg, ranks_per_node=6)
        assert np.array_equal(bufs.to_host(), ref.bufs) and bufs.guards_intact()
        assert np.array_equal(counts.cpu().numpy(), ref.col("len"))

"""One process per GPU without GPUs: the phase loop of paper_1603_06809_b200.sharded run by two and
three `gloo` ranks on CPU.  Each process owns the rank buffers of "its GPU" inside one block of shared
memory (standing in for peer-mapped device memory) and, where the GPU path would launch a kernel,
replays the partition's hop list of that (phase, GPU) with plain copies.  The barrier after every
phase is all that orders the processes; the buffers must come out equal to the oracle's."""
import os
import sys
from multiprocessing import shared_memory

import numpy as np
import pytest
import torch.multiprocessing as mp

from helpers import ROOT


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, shm_name, P, root, n, variant, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from paper_1603_06809_b200 import bcast as B
    from paper_1603_06809_b200 import sharded
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    shm = shared_memory.SharedMemory(name=shm_name)
    bufs = np.ndarray((P, n), dtype=np.uint8, buffer=shm.buf)
    plan = B.bcast_plan(P, root, n, variant)
    shard = B.bcast_shard_create(plan, world)
    x = B.bcast_plan_xfers(plan)
    S = B.bcast_plan_scatter_size(plan)
    mine = sharded.owned_ranks(shard, rank)
    calls = []

    def exec_phase(phase):                       # stands in for this GPU's kernel of the phase
        calls.append(phase)
        for c in range(P):
            lo, hi = min(c * S, n), min((c + 1) * S, n)
            for m in B.bcast_shard_hops(shard, phase, rank, c):
                assert int(x["dst_rank"][m]) in mine
                bufs[int(x["dst_rank"][m]), lo:hi] = bufs[int(x["src_rank"][m]), lo:hi]

    phases = sharded.run_phases(shard, rank, [], exec_phase, lambda: None, dist.barrier)
    assert calls == list(range(phases))
    dist.barrier()
    out.put((rank, phases, mine))
    shm.close()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,P,root,n,variant", [(2, 12, 5, 12 * 700 + 5, 1), (2, 8, 0, 8 * 1024, 0), (3, 10, 7, 10 * 333, 1),
                                                    (2, 16, 3, 16 * 100 + 1, 2)])
def test_phase_loop_on_gloo_ranks_matches_the_oracle(oracle, world, P, root, n, variant):
    sys.path.insert(0, ROOT)
    from paper_1603_06809_b200 import workloads as W
    msg = W.message_bytes(31 + P, n)
    ref = oracle.simulate(P, root, n, variant, message=msg)
    shm = shared_memory.SharedMemory(create=True, size=P * n)
    try:
        bufs = np.ndarray((P, n), dtype=np.uint8, buffer=shm.buf)
        for k in range(P):
            bufs[k, :] = W.poison_byte(k)
        bufs[root, :] = msg
        ctx = mp.get_context("spawn")
        out = ctx.Queue()
        port = _free_port()
        procs = [ctx.Process(target=_rank_main, args=(r, world, port, shm.name, P, root, n, variant, out)) for r in range(world)]
        for p in procs:
            p.start()
        got = sorted(out.get(timeout=180) for _ in range(world))
        for p in procs:
            p.join(timeout=60)
            assert p.exitcode == 0
        assert np.array_equal(bufs, ref.bufs)
        owned = sorted(r for _, _, mine in got for r in mine)
        assert owned == list(range(P))                       # every rank has exactly one owner
        assert len({phases for _, phases, _ in got}) == 1    # all processes ran the same number of phases
        del bufs
    finally:
        shm.close()
        shm.unlink()

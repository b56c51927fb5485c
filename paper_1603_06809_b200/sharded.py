"""One process per GPU: the P ranks of a broadcast spread over the processes of a torch.distributed
group, every process owning the rank buffers of its GPU.

Host-side plumbing only.  The partition, the phases and the kernels are the library's
(``bcast_shard_*`` in ``include/bcast.h``); this module decides nothing about the method.  What it
does: allocate the local rank buffers, exchange handles so that every process can read the others'
buffers (CUDA IPC mappings; peer loads over NVLink where the GPUs differ), and run the phases in
order with a barrier after each one -- phase k+1 of any GPU may only start when phase k of every GPU
has completed.  No kernel waits for another kernel and no collective moves data.
"""
from __future__ import annotations

from typing import Callable, Sequence

from . import bcast as B


def owned_ranks(shard: B.Shard, gpu: int) -> list[int]:
    """Absolute ranks whose buffers live on GPU ``gpu`` of the partition."""
    return [r for r, g in enumerate(B.bcast_shard_rank_gpu(shard)) if g == gpu]


def run_phases(shard: B.Shard, gpu: int, rank_ptrs: Sequence[int], exec_phase: Callable[[int], None],
               wait_local: Callable[[], None], barrier: Callable[[], None]) -> int:
    """The phase loop of one process.  ``exec_phase(phase)`` enqueues this GPU's kernel of that phase,
    ``wait_local()`` waits for it, ``barrier()`` returns once every process has called it.  Returns
    the number of phases.  A barrier opens the loop: nobody starts before every process (the root's
    owner in particular, which has just put the message in place) is ready."""
    del rank_ptrs  # the callables hold what they need; kept in the signature for symmetry with the C entry point
    barrier()
    phases = B.bcast_shard_num_phases(shard)
    for phase in range(phases):
        exec_phase(phase)
        wait_local()
        barrier()
    return phases


class ShardedBroadcast:
    """One process's end of a broadcast whose ranks are spread over ``world`` GPUs.

    ``device``: the torch CUDA device of this process.  ``group_rank`` / ``world``: this process's
    index and the number of processes; process g owns GPU g of the partition.  ``all_gather_object``:
    a callable like ``torch.distributed.all_gather_object`` bound to the group; ``barrier`` likewise.
    """

    def __init__(self, P: int, root: int, nbytes: int, variant: int, group_rank: int, world: int, device,
                 all_gather_object, barrier):
        import torch
        self.torch = torch
        self.P, self.root, self.nbytes, self.gpu, self.world = P, root, nbytes, group_rank, world
        self.device = torch.device(device)
        self.barrier = barrier
        self.plan = B.bcast_plan(P, root, nbytes, variant)
        self.shard = B.bcast_shard_create(self.plan, world)
        self.mine = owned_ranks(self.shard, self.gpu)
        self.stride = (nbytes + 511) // 256 * 256
        with torch.cuda.device(self.device):
            self.local = torch.empty((max(1, len(self.mine)), self.stride), dtype=torch.uint8, device=self.device)
        # every process learns how to reach every other process's buffers
        handle = self.local.untyped_storage()._share_cuda_()
        handles = [None] * world
        all_gather_object(handles, (self.gpu, handle, self.local.storage_offset()))
        self._peers = {}
        base = {}
        for g, h, off in handles:
            if g == self.gpu:
                base[g] = self.local.data_ptr()
            else:
                storage = torch.UntypedStorage._new_shared_cuda(*h)
                self._peers[g] = storage                      # keeps the mapping open
                base[g] = storage.data_ptr() + off
        owner = B.bcast_shard_rank_gpu(self.shard)
        index = {}
        for g in range(world):
            for i, r in enumerate(owned_ranks(self.shard, g)):
                index[r] = i
        self.rank_ptrs = [base[int(owner[r])] + index[r] * self.stride for r in range(P)]
        self.stream = torch.cuda.current_stream(self.device)

    def local_view(self, rank: int):
        """The buffer of an owned rank (first nbytes bytes)."""
        return self.local[self.mine.index(rank), : self.nbytes]

    def owns(self, rank: int) -> bool:
        return rank in self.mine

    def run(self, device_msg_bytes=None) -> int:
        """One broadcast: all phases, with a barrier after each.  Returns the number of phases."""
        def exec_phase(phase):
            B.bcast_shard_exec_phase(self.shard, self.rank_ptrs, phase, self.gpu, self.stream, device_msg_bytes)
        return run_phases(self.shard, self.gpu, self.rank_ptrs, exec_phase, self.stream.synchronize, self.barrier)

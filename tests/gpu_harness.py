"""Harness of the GPU parity tests: rank buffers with guard zones, one broadcast through the
C ABI, comparison with the oracle.  Holds no arithmetic of the method."""
import numpy as np
import torch

from paper_1603_06809_b200 import bcast as B
from paper_1603_06809_b200 import workloads as W

GUARD = 256           # bytes of canary before and after every rank buffer
CANARY = 0xC3


class RankBuffers:
    """P device buffers of nbytes each, every one inside its own allocation between two guard
    zones.  The root holds the message, the others a rank-dependent poison."""

    def __init__(self, P, root, nbytes, message, device="cuda:0", shift=0):
        self.P, self.root, self.nbytes = P, root, nbytes
        self.raw, self.view = [], []
        msg = torch.from_numpy(np.ascontiguousarray(message)).to(device) if nbytes else None
        self.message = msg
        for k in range(P):
            t = torch.full((GUARD + shift + nbytes + GUARD,), CANARY, dtype=torch.uint8, device=device)
            v = t[GUARD + shift: GUARD + shift + nbytes]
            if nbytes:
                if k == root:
                    v.copy_(msg)
                else:
                    v.fill_(W.poison_byte(k))
            self.raw.append(t)
            self.view.append(v)
        self.shift = shift

    def pointers(self):
        return [t.data_ptr() + GUARD + self.shift for t in self.raw]

    def reset(self):
        for k in range(self.P):
            if k != self.root and self.nbytes:
                self.view[k].fill_(W.poison_byte(k))

    def guards_intact(self):
        for t in self.raw:
            lo = t[: GUARD + self.shift]
            hi = t[GUARD + self.shift + self.nbytes:]
            if not (bool((lo == CANARY).all()) and bool((hi == CANARY).all())):
                return False
        return True

    def all_equal_message(self):
        if not self.nbytes:
            return True
        return all(torch.equal(v, self.message) for v in self.view)

    def to_host(self):
        out = np.empty((self.P, self.nbytes), dtype=np.uint8)
        for k in range(self.P):
            if self.nbytes:
                out[k] = self.view[k].cpu().numpy()
        return out


def run_broadcast(P, root, nbytes, variant, mode, message, shift=0, repeats=1, ranks_per_node=0):
    """Plan + execute through the C ABI on cuda:0; returns (plan, RankBuffers) after a sync."""
    bufs = RankBuffers(P, root, nbytes, message, shift=shift)
    plan = B.bcast_plan_smp(P, root, nbytes, variant, ranks_per_node) if ranks_per_node else B.bcast_plan(P, root, nbytes, variant)
    stream = torch.cuda.current_stream()
    for rep in range(repeats):
        if rep:
            bufs.reset()
        B.bcast_exec_mode(bufs.pointers(), plan, stream, mode)
    torch.cuda.synchronize()
    return plan, bufs

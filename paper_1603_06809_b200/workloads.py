"""Seeded synthetic workloads: the broadcast configurations and the root's message bytes.

This module holds no arithmetic of the broadcast method.  It only names the problem sizes and
draws the message content, so that the CUDA path, the tests and the CPU oracle can all be fed
the same bytes.  The paper's workload is a micro-benchmark over byte messages whose content does
not matter (Section V); uniform random bytes stand in for it.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

KiB, MiB = 1 << 10, 1 << 20
BASE_SEED = 160306809


@dataclass(frozen=True)
class Workload:
    name: str
    P: int          # number of virtual ranks
    root: int
    nbytes: int     # message size
    seed: int

    @property
    def total_bytes(self) -> int:
        return self.P * self.nbytes


#: the four single-point configurations
CFG1 = Workload("P8_root0_1MiB", 8, 0, 1 * MiB, BASE_SEED + 1)
CFG2 = Workload("P12_root5_256KiB", 12, 5, 256 * KiB, BASE_SEED + 2)
CFG3 = Workload("P64_root17_16MiB+13", 64, 17, 16 * MiB + 13, BASE_SEED + 3)
CFG4 = Workload("P100_root63_64MiB", 100, 63, 64 * MiB, BASE_SEED + 4)

SWEEP_P = (2, 3, 7, 16, 24, 33, 128, 255, 256)
SWEEP_NBYTES = (12 * KiB, 512 * KiB, 4 * MiB, 32 * MiB, 128 * MiB)
SWEEP_CAP_BYTES = 64 * 10**9


def cfg2_all_roots() -> list[Workload]:
    """Configuration 2 with every root 0..11."""
    return [Workload(f"P12_root{r}_256KiB", 12, r, 256 * KiB, BASE_SEED + 2) for r in range(12)]


def sweep() -> list[Workload]:
    """Configuration 5: P x nbytes grid, root = P-1, total rank-buffer bytes capped."""
    out = []
    for P in SWEEP_P:
        for n in SWEEP_NBYTES:
            if P * n <= SWEEP_CAP_BYTES:
                out.append(Workload(f"sweep_P{P}_{n}B", P, P - 1, n, BASE_SEED + 5))
    return out


def message_bytes(seed: int, nbytes: int) -> np.ndarray:
    """The root's message: ``nbytes`` uniform random uint8 from a seeded counter-based generator."""
    rng = np.random.Generator(np.random.Philox(key=seed))
    return rng.integers(0, 256, size=nbytes, dtype=np.uint8)


def poison_byte(rank: int) -> int:
    """Fill value for a non-root buffer before the broadcast; differs from rank to rank."""
    return (0x5A + 29 * rank) & 0xFF


# ---- the paper's own experiment shapes (Section V), as a second workload set
#: Experiment A: long messages, power-of-two process counts (Fig. 6)
PAPER_A_P = (16, 64, 256)
PAPER_A_NBYTES = (524288, 1 * MiB, 2 * MiB, 4 * MiB, 8 * MiB, 16 * MiB, 30_000_000)
#: Experiment B: non-power-of-two process counts at the two MPICH thresholds and 1 MiB (Fig. 7)
PAPER_B_P = (9, 17, 33, 65, 129)
PAPER_B_NBYTES = (12288, 524287, 1048576)
#: Experiment C: 129 processes, 12288 ... 2,560,000 bytes (Fig. 8)
PAPER_C_P = 129
PAPER_C_NBYTES = (12288, 65536, 262144, 524288, 1048576, 2_560_000)


def paper_experiments() -> list[Workload]:
    """Message sizes and process counts of the paper's three experiments; root 0 as in a plain
    micro-benchmark.  Sizes between the end points that the paper names are a geometric fill."""
    out = []
    for P in PAPER_A_P:
        out += [Workload(f"paperA_P{P}_{n}B", P, 0, n, BASE_SEED + 6) for n in PAPER_A_NBYTES]
    for P in PAPER_B_P:
        out += [Workload(f"paperB_P{P}_{n}B", P, 0, n, BASE_SEED + 7) for n in PAPER_B_NBYTES]
    out += [Workload(f"paperC_P{PAPER_C_P}_{n}B", PAPER_C_P, 0, n, BASE_SEED + 8) for n in PAPER_C_NBYTES]
    return out

"""ctypes front end of the CPU oracle (oracle/bcast_oracle.c).

TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT: only the tests, the smoke check and the
CPU-baseline / reference legs of the benchmark may import this module.  It imports nothing
from the CUDA package and the CUDA package imports nothing from here.

The C file is compiled with gcc on first use into ``oracle/_build``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import time
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bcast_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libbcast_oracle.so")

NATIVE, TUNED, DOUBLING = 0, 1, 2
SCATTER, RING = 0, 1
NODE_FIRST, NODE_LAST = 2, 3     # node-aware broadcast only: tree broadcast in the root's node / in the other nodes
SEND_ONLY, RECV_ONLY = 0, 1

#: column names of the schedule array returned by :func:`simulate`
FIELDS = ("phase", "step", "src", "dst", "chunk", "nchunks", "offset", "len", "dep")

ERRORS = {
    -1: "bad argument", -2: "out of memory", -3: "schedule capacity exceeded",
    -4: "a sender did not hold what it sends", -5: "send without matching receive",
    -7: "a step reads what it writes",
    -8: "a process misses a chunk at the end", -9: "a buffer differs from the root's message",
}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than the source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        os.makedirs(os.path.dirname(_LIB), exist_ok=True)
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-Wall", "-Wextra", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _bind(path: str):
    """Load a build of the oracle and declare its signatures."""
    lib = ctypes.CDLL(path)
    u64p = ctypes.POINTER(ctypes.c_uint64)
    lib.oracle_bcast_simulate.restype = ctypes.c_int
    lib.oracle_bcast_simulate.argtypes = [
        ctypes.c_int, ctypes.c_int, ctypes.c_uint64, ctypes.c_int, ctypes.POINTER(ctypes.c_void_p),
        ctypes.POINTER(ctypes.c_int64), ctypes.c_int64, ctypes.POINTER(ctypes.c_int64),
        u64p, u64p, u64p, u64p]
    lib.oracle_bcast_simulate_smp.restype = ctypes.c_int
    lib.oracle_bcast_simulate_smp.argtypes = [
        ctypes.c_int, ctypes.c_int, ctypes.c_uint64, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_void_p),
        ctypes.POINTER(ctypes.c_int64), ctypes.c_int64, ctypes.POINTER(ctypes.c_int64),
        u64p, u64p, u64p, u64p]
    lib.oracle_bcast_scatter_size.restype = ctypes.c_uint64
    lib.oracle_bcast_scatter_size.argtypes = [ctypes.c_int, ctypes.c_uint64]
    lib.oracle_bcast_step_flag.restype = ctypes.c_int
    lib.oracle_bcast_step_flag.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


def use_build(path: str | None):
    """Tests only: route all calls to another build of the oracle (a deliberately broken copy, to
    show that the pins notice); ``None`` switches back to the real one."""
    global _lib
    _lib = _bind(path) if path else None


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle check failed ({code}): {ERRORS.get(code, '?')}")
        self.code = code


@dataclass
class OracleResult:
    P: int
    root: int
    nbytes: int
    variant: int
    scatter_size: int
    schedule: np.ndarray      # (N, 9) int64, columns = FIELDS, canonical order
    bytes_sent: np.ndarray    # (2, P) uint64: [phase, absolute rank]
    bytes_recv: np.ndarray
    msgs_sent: np.ndarray
    msgs_recv: np.ndarray
    bufs: np.ndarray | None   # (P, nbytes) uint8 after the broadcast, or None (schedule only)
    seconds: float            # wall time of the simulation call alone

    def col(self, name: str) -> np.ndarray:
        return self.schedule[:, FIELDS.index(name)]

    def phase_rows(self, phase: int) -> np.ndarray:
        return self.schedule[self.col("phase") == phase]


def scatter_size(P: int, nbytes: int) -> int:
    return int(_load().oracle_bcast_scatter_size(P, nbytes))


def step_flags(P: int) -> list[tuple[int, int]]:
    """(step, flag) of the tuned ring for every relative rank 0..P-1; flag is SEND_ONLY or RECV_ONLY."""
    step, flag = (ctypes.c_int * P)(), (ctypes.c_int * P)()
    rc = _load().oracle_bcast_step_flag(P, step, flag)
    if rc:
        raise OracleError(rc)
    return list(zip(step, flag))


def step_flag(P: int, rel_rank: int) -> tuple[int, int]:
    """(step, flag) of one relative rank (see :func:`step_flags`)."""
    return step_flags(P)[rel_rank]


def capacity(P: int) -> int:
    """Upper bound on the number of messages: P-1 scatter messages and P(P-1) ring messages."""
    return max(1, (P - 1) + P * (P - 1))


def simulate(P: int, root: int, nbytes: int, variant: int, message: np.ndarray | None = None,
             bufs: np.ndarray | None = None, ranks_per_node: int = 0) -> OracleResult:
    """Run the simulated broadcast.

    ``message``: uint8 array of ``nbytes`` (the root's data) -> per-rank buffers are created here,
    non-root ones filled with a rank-dependent poison.  ``bufs``: a caller-made (P, nbytes) uint8
    array used in place (the caller has put the message into ``bufs[root]``).  Neither: schedule
    and counters only, no data moved.  ``ranks_per_node`` >= 1: the node-aware broadcast (tree
    broadcast in the root's node, scatter-ring between the node leaders, tree broadcast in the
    other nodes); the counter arrays then have four phases.
    """
    lib = _load()
    if bufs is None and message is not None:
        message = np.ascontiguousarray(message, dtype=np.uint8)
        assert message.shape == (nbytes,)
        bufs = np.empty((P, nbytes), dtype=np.uint8)
        for k in range(P):
            bufs[k, :] = (0xA5 ^ (k * 37 + 11)) & 0xFF
        bufs[root, :] = message
    ptrs = None
    if bufs is not None:
        assert bufs.dtype == np.uint8 and bufs.shape == (P, nbytes) and bufs.flags.c_contiguous
        base = bufs.ctypes.data
        ptrs = (ctypes.c_void_p * P)(*[base + k * nbytes for k in range(P)])
    cap = capacity(P)
    sched = np.zeros((cap, len(FIELDS)), dtype=np.int64)
    nsched = ctypes.c_int64(0)
    nphases = 4 if ranks_per_node else 2
    cnt = [np.zeros((nphases, P), dtype=np.uint64) for _ in range(4)]
    u64p = ctypes.POINTER(ctypes.c_uint64)
    t0 = time.perf_counter()
    if ranks_per_node:
        rc = lib.oracle_bcast_simulate_smp(
            P, root, nbytes, variant, ranks_per_node, ptrs,
            sched.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), cap, ctypes.byref(nsched),
            *[c.ctypes.data_as(u64p) for c in cnt])
    else:
        rc = lib.oracle_bcast_simulate(
            P, root, nbytes, variant, ptrs,
            sched.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), cap, ctypes.byref(nsched),
            *[c.ctypes.data_as(u64p) for c in cnt])
    dt = time.perf_counter() - t0
    if rc:
        raise OracleError(rc)
    nchunks = -(-P // ranks_per_node) if ranks_per_node else P
    return OracleResult(P=P, root=root, nbytes=nbytes, variant=variant,
                        scatter_size=scatter_size(nchunks, nbytes),
                        schedule=sched[: nsched.value].copy(),
                        bytes_sent=cnt[0], bytes_recv=cnt[1], msgs_sent=cnt[2], msgs_recv=cnt[3],
                        bufs=bufs, seconds=dt)


# ---- the all-cores CPU baseline: the oracle's schedule replayed by a team of threads
_SRC_MT = os.path.join(_HERE, "bcast_oracle_mt.c")
_LIB_MT = os.path.join(_HERE, "_build", "libbcast_oracle_mt.so")
_lib_mt = None


def build_mt(force: bool = False) -> str:
    """Compile oracle/bcast_oracle_mt.c (pthreads) if missing or stale."""
    if force or not os.path.exists(_LIB_MT) or os.path.getmtime(_LIB_MT) < os.path.getmtime(_SRC_MT):
        os.makedirs(os.path.dirname(_LIB_MT), exist_ok=True)
        tmp = _LIB_MT + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-Wall", "-Wextra", "-pthread", "-shared", "-fPIC", "-o", tmp, _SRC_MT])
        os.replace(tmp, _LIB_MT)
    return _LIB_MT


def replay_mt(P: int, schedule: np.ndarray, bufs: np.ndarray, nthreads: int) -> float:
    """Perform the messages of ``schedule`` (as returned by :func:`simulate`) on ``bufs`` ((P, nbytes)
    uint8, the root's row holding the message) with ``nthreads`` threads, step by step with a barrier
    after every step.  Returns the wall time in seconds.  Only the benchmark's all-cores CPU baseline
    and the test that compares its buffers with the single-threaded oracle's use this."""
    global _lib_mt
    if _lib_mt is None:
        _lib_mt = ctypes.CDLL(build_mt())
        _lib_mt.oracle_bcast_replay_mt.restype = ctypes.c_int
        _lib_mt.oracle_bcast_replay_mt.argtypes = [
            ctypes.c_int, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_int64), ctypes.c_int64,
            ctypes.c_int, ctypes.POINTER(ctypes.c_double)]
    assert bufs.dtype == np.uint8 and bufs.ndim == 2 and bufs.shape[0] == P and bufs.flags.c_contiguous
    sched = np.ascontiguousarray(schedule, dtype=np.int64)
    assert sched.ndim == 2 and sched.shape[1] == len(FIELDS)
    nbytes = bufs.shape[1]
    if len(sched):
        assert int((sched[:, FIELDS.index("offset")] + sched[:, FIELDS.index("len")]).max()) <= nbytes
    base = bufs.ctypes.data
    ptrs = (ctypes.c_void_p * P)(*[base + k * nbytes for k in range(P)])
    seconds = ctypes.c_double(0.0)
    rc = _lib_mt.oracle_bcast_replay_mt(P, ptrs, sched.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), len(sched),
                                        nthreads, ctypes.byref(seconds))
    if rc:
        raise OracleError(rc)
    return seconds.value

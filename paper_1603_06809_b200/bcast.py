"""ctypes binding of ``include/bcast.h``: same names, argument marshalling only.

Every function here forwards to the C-ABI entry point of the same name in ``libbcast_b200.so``;
no step of the broadcast is computed in Python.  Importing this module fails loudly when the
library is missing: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libbcast_b200.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_1603_06809_b200.build` "
        "(nvcc, sm_100a).  There is no CPU fallback.")
_lib = ctypes.CDLL(_LIB_PATH)

BCAST_MAX_RANKS = 1024
BCAST_NATIVE, BCAST_TUNED, BCAST_DOUBLING = 0, 1, 2
BCAST_PHASE_SCATTER, BCAST_PHASE_RING, BCAST_PHASE_NODE_FIRST, BCAST_PHASE_NODE_LAST = 0, 1, 2, 3
BCAST_OK, BCAST_ERR_INVAL, BCAST_ERR_NOMEM, BCAST_ERR_CUDA, BCAST_ERR_CAPACITY, BCAST_ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
BCAST_STATIC_SCRATCH_BYTES = 2 << 20
BCAST_EXEC_WALK, BCAST_EXEC_STEPS, BCAST_EXEC_GRAPH, BCAST_EXEC_WALK_PLAN_ORDER = 0, 1, 2, 3
BCAST_EXEC_WALK_BULK, BCAST_EXEC_AUTO = 4, 5

#: numpy view of ``bcast_xfer_t`` (48 bytes)
XFER_DTYPE = np.dtype([
    ("phase", "<i4"), ("step", "<i4"), ("src_rank", "<i4"), ("dst_rank", "<i4"),
    ("chunk", "<i4"), ("nchunks", "<i4"), ("offset", "<u8"), ("len", "<u8"), ("dep", "<i8")], align=True)
assert XFER_DTYPE.itemsize == 48

#: every symbol ``include/bcast.h`` declares
SYMBOLS = (
    "bcast_plan", "bcast_plan_smp", "bcast_plan_free", "bcast_plan_num_ranks", "bcast_plan_root", "bcast_plan_variant",
    "bcast_plan_ranks_per_node", "bcast_plan_num_chunks",
    "bcast_plan_nbytes", "bcast_plan_scatter_size", "bcast_plan_num_xfers", "bcast_plan_num_steps",
    "bcast_plan_xfers", "bcast_plan_step_begin", "bcast_plan_bytes_sent", "bcast_plan_bytes_recv",
    "bcast_plan_msgs_sent", "bcast_plan_msgs_recv", "bcast_plan_total_bytes", "bcast_plan_walk_order",
    "bcast_plan_walk_pairing", "bcast_plan_walk_slices", "bcast_exec_traced", "bcast_exec",
    "bcast_shard_create", "bcast_shard_free", "bcast_shard_num_gpus", "bcast_shard_num_phases", "bcast_shard_rank_gpu",
    "bcast_shard_msg_gpu", "bcast_shard_msg_phase", "bcast_shard_crossing_bytes", "bcast_shard_crossing_msgs",
    "bcast_shard_hops", "bcast_shard_exec", "bcast_shard_exec_phase",
    "bcast_exec_mode", "bcast_exec_host", "bcast_exec_static", "bcast_exec_status", "bcast_exec_num_launches", "bcast_strerror",
    "bcast_last_cuda_error",
)

_vp, _i, _i32, _i64, _u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64
_vpp = ctypes.POINTER(ctypes.c_void_p)
_sig = {
    "bcast_plan": (_i, [_i, _i, _u64, _i, _vpp]),
    "bcast_plan_smp": (_i, [_i, _i, _u64, _i, _i, _vpp]),
    "bcast_plan_ranks_per_node": (_i32, [_vp]), "bcast_plan_num_chunks": (_i32, [_vp]),
    "bcast_plan_free": (None, [_vp]),
    "bcast_plan_num_ranks": (_i32, [_vp]), "bcast_plan_root": (_i32, [_vp]), "bcast_plan_variant": (_i32, [_vp]),
    "bcast_plan_nbytes": (_u64, [_vp]), "bcast_plan_scatter_size": (_u64, [_vp]),
    "bcast_plan_num_xfers": (_i64, [_vp]), "bcast_plan_num_steps": (_i32, [_vp]),
    "bcast_plan_xfers": (_vp, [_vp]), "bcast_plan_step_begin": (_vp, [_vp]),
    "bcast_plan_bytes_sent": (_vp, [_vp, _i]), "bcast_plan_bytes_recv": (_vp, [_vp, _i]),
    "bcast_plan_msgs_sent": (_vp, [_vp, _i]), "bcast_plan_msgs_recv": (_vp, [_vp, _i]),
    "bcast_plan_total_bytes": (_u64, [_vp]),
    "bcast_plan_walk_order": (_i64, [_vp, _i, _i, ctypes.POINTER(ctypes.c_int64), _i64]),
    "bcast_plan_walk_pairing": (_i64, [_vp, _i, ctypes.POINTER(ctypes.c_int64), _i64]),
    "bcast_plan_walk_slices": (_i64, [_vp, _i, ctypes.POINTER(ctypes.c_int64), _i64]),
    "bcast_exec_traced": (_i, [_vpp, _vp, _vp, _i, _vp]),
    "bcast_exec": (_i, [_vpp, _vp, _vp]),
    "bcast_shard_create": (_i, [_vp, _i, ctypes.POINTER(ctypes.c_int32), _vpp]),
    "bcast_shard_free": (None, [_vp]),
    "bcast_shard_num_gpus": (_i32, [_vp]), "bcast_shard_num_phases": (_i32, [_vp]),
    "bcast_shard_rank_gpu": (_vp, [_vp]), "bcast_shard_msg_gpu": (_vp, [_vp]), "bcast_shard_msg_phase": (_vp, [_vp, _i]),
    "bcast_shard_crossing_bytes": (_u64, [_vp]), "bcast_shard_crossing_msgs": (_i64, [_vp]),
    "bcast_shard_hops": (_i64, [_vp, _i, _i, _i, ctypes.POINTER(ctypes.c_int64), _i64]),
    "bcast_shard_exec": (_i, [_vp, _vpp, ctypes.POINTER(ctypes.c_int), _vpp, _vp]),
    "bcast_shard_exec_phase": (_i, [_vp, _vpp, _i, _i, _vp, _vp]),
    "bcast_exec_mode": (_i, [_vpp, _vp, _vp, _i]),
    "bcast_exec_host": (_i, [_vpp, _vp, _vp, _i, _vp, _vpp]),
    "bcast_exec_static": (_i, [_vpp, _vp, _vp]),
    "bcast_exec_status": (_i, [_vp]),
    "bcast_exec_num_launches": (_i64, [_vp, _i]),
    "bcast_strerror": (ctypes.c_char_p, [_i]),
    "bcast_last_cuda_error": (_i, []),
}
for _name, (_res, _args) in _sig.items():
    _f = getattr(_lib, _name)
    _f.restype, _f.argtypes = _res, _args


class BcastError(RuntimeError):
    def __init__(self, code: int, where: str):
        msg = _lib.bcast_strerror(code).decode()
        if code == BCAST_ERR_CUDA:
            msg += f" (cudaError {_lib.bcast_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{code}]")
        self.code = code


def _check(code: int, where: str) -> None:
    if code != BCAST_OK:
        raise BcastError(code, where)


def _view(ptr, count, dtype):
    """Copy `count` items of `dtype` from a library-owned host pointer into a numpy array."""
    if not ptr or count == 0:
        return np.zeros(0, dtype=dtype)
    buf = (ctypes.c_char * (count * np.dtype(dtype).itemsize)).from_address(ptr)
    return np.frombuffer(buf, dtype=dtype, count=count).copy()


class Plan:
    """Owner of a ``bcast_plan_t*``; the handle is released when the object is collected."""

    def __init__(self, handle: int):
        self._h = ctypes.c_void_p(handle)

    @property
    def handle(self) -> ctypes.c_void_p:
        if not self._h:
            raise ValueError("plan already freed")
        return self._h

    def free(self) -> None:
        if self._h:
            _lib.bcast_plan_free(self._h)
            self._h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def bcast_plan(P: int, root: int, nbytes: int, variant: int) -> Plan:
    out = ctypes.c_void_p(None)
    _check(_lib.bcast_plan(P, root, nbytes, variant, ctypes.byref(out)), "bcast_plan")
    return Plan(out.value)


def bcast_plan_smp(P: int, root: int, nbytes: int, variant: int, ranks_per_node: int) -> Plan:
    out = ctypes.c_void_p(None)
    _check(_lib.bcast_plan_smp(P, root, nbytes, variant, ranks_per_node, ctypes.byref(out)), "bcast_plan_smp")
    return Plan(out.value)


def bcast_plan_free(plan: Plan) -> None:
    plan.free()


def bcast_plan_num_ranks(plan: Plan) -> int: return _lib.bcast_plan_num_ranks(plan.handle)
def bcast_plan_root(plan: Plan) -> int: return _lib.bcast_plan_root(plan.handle)
def bcast_plan_variant(plan: Plan) -> int: return _lib.bcast_plan_variant(plan.handle)
def bcast_plan_ranks_per_node(plan: Plan) -> int: return _lib.bcast_plan_ranks_per_node(plan.handle)
def bcast_plan_num_chunks(plan: Plan) -> int: return _lib.bcast_plan_num_chunks(plan.handle)
def bcast_plan_nbytes(plan: Plan) -> int: return _lib.bcast_plan_nbytes(plan.handle)
def bcast_plan_scatter_size(plan: Plan) -> int: return _lib.bcast_plan_scatter_size(plan.handle)
def bcast_plan_num_xfers(plan: Plan) -> int: return _lib.bcast_plan_num_xfers(plan.handle)
def bcast_plan_num_steps(plan: Plan) -> int: return _lib.bcast_plan_num_steps(plan.handle)
def bcast_plan_total_bytes(plan: Plan) -> int: return _lib.bcast_plan_total_bytes(plan.handle)


def bcast_plan_xfers(plan: Plan) -> np.ndarray:
    """The schedule as a structured array (copy), fields as in ``bcast_xfer_t``."""
    return _view(_lib.bcast_plan_xfers(plan.handle), bcast_plan_num_xfers(plan), XFER_DTYPE)


def bcast_plan_step_begin(plan: Plan) -> np.ndarray:
    n = bcast_plan_num_steps(plan)
    return _view(_lib.bcast_plan_step_begin(plan.handle), n + 1, np.int64)


def _counter(fn, plan: Plan, phase: int) -> np.ndarray:
    ptr = fn(plan.handle, phase)
    if not ptr:
        raise BcastError(BCAST_ERR_INVAL, fn.__name__)
    return _view(ptr, bcast_plan_num_ranks(plan), np.uint64)


def bcast_plan_bytes_sent(plan: Plan, phase: int) -> np.ndarray: return _counter(_lib.bcast_plan_bytes_sent, plan, phase)
def bcast_plan_bytes_recv(plan: Plan, phase: int) -> np.ndarray: return _counter(_lib.bcast_plan_bytes_recv, plan, phase)
def bcast_plan_msgs_sent(plan: Plan, phase: int) -> np.ndarray: return _counter(_lib.bcast_plan_msgs_sent, plan, phase)
def bcast_plan_msgs_recv(plan: Plan, phase: int) -> np.ndarray: return _counter(_lib.bcast_plan_msgs_recv, plan, phase)


def bcast_plan_walk_order(plan: Plan, chunk: int, mode: int = BCAST_EXEC_WALK) -> np.ndarray:
    """Indices into the schedule of the messages that move chunk ``chunk``, in the order the WALK
    executor performs them."""
    n = _lib.bcast_plan_walk_order(plan.handle, chunk, mode, None, 0)
    if n < 0:
        raise BcastError(int(n), "bcast_plan_walk_order")
    out = np.zeros(int(n), dtype=np.int64)
    if n:
        got = _lib.bcast_plan_walk_order(plan.handle, chunk, mode,
                                         out.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), int(n))
        assert got == n
    return out


def _fill_i64(fn, plan: Plan, arg: int, width: int, where: str) -> np.ndarray:
    """Two-call protocol of the list-returning entry points: size first, then the entries."""
    n = fn(plan.handle, arg, None, 0)
    if n < 0:
        raise BcastError(int(n), where)
    out = np.zeros((int(n), width), dtype=np.int64)
    if n:
        got = fn(plan.handle, arg, out.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), int(n))
        assert got == n
    return out


def bcast_plan_walk_pairing(plan: Plan, chunk: int) -> np.ndarray:
    """(slots, 2) array: per slot the message of chunk ``chunk`` and that of chunk ``chunk + 1``
    (indices into the schedule, -1 where the slot has none)."""
    return _fill_i64(_lib.bcast_plan_walk_pairing, plan, chunk, 2, "bcast_plan_walk_pairing")


def bcast_plan_walk_slices(plan: Plan, words: int) -> np.ndarray:
    """(slices, 3) array: segment index, kind (0 whole / 1 ragged / 2 dual), (lower) chunk."""
    return _fill_i64(_lib.bcast_plan_walk_slices, plan, words, 3, "bcast_plan_walk_slices")


def _ptr_array(items, what: str):
    """A C array of pointers from ints, objects with ``data_ptr()`` (torch tensors) or None."""
    vals = []
    for x in items:
        if x is None:
            vals.append(None)
        elif hasattr(x, "data_ptr"):
            vals.append(x.data_ptr())
        else:
            vals.append(int(x))
    return (ctypes.c_void_p * len(vals))(*vals)


def _stream_ptr(stream) -> ctypes.c_void_p:
    if stream is None:
        return ctypes.c_void_p(None)
    return ctypes.c_void_p(int(getattr(stream, "cuda_stream", stream)))


def bcast_exec(rank_bufs, plan: Plan, stream=None) -> None:
    """``rank_bufs``: P device pointers (ints) or torch CUDA tensors; ``stream``: a
    ``torch.cuda.Stream``, a raw ``cudaStream_t`` value, or None for the default stream."""
    if len(rank_bufs) != bcast_plan_num_ranks(plan):
        raise BcastError(BCAST_ERR_INVAL, "bcast_exec (len(rank_bufs) != P)")
    _check(_lib.bcast_exec(_ptr_array(rank_bufs, "rank_bufs"), plan.handle, _stream_ptr(stream)), "bcast_exec")


def bcast_exec_mode(rank_bufs, plan: Plan, stream=None, mode: int = BCAST_EXEC_AUTO) -> None:
    if len(rank_bufs) != bcast_plan_num_ranks(plan):
        raise BcastError(BCAST_ERR_INVAL, "bcast_exec_mode (len(rank_bufs) != P)")
    _check(_lib.bcast_exec_mode(_ptr_array(rank_bufs, "rank_bufs"), plan.handle, _stream_ptr(stream), mode),
           "bcast_exec_mode")


def bcast_exec_traced(rank_bufs, plan: Plan, stream, mode: int, device_msg_bytes) -> None:
    """``device_msg_bytes``: device pointer (int) or CUDA tensor of ``num_xfers`` zeroed 64-bit
    counters; the kernels add the bytes they store for every message."""
    if len(rank_bufs) != bcast_plan_num_ranks(plan):
        raise BcastError(BCAST_ERR_INVAL, "bcast_exec_traced (len(rank_bufs) != P)")
    ptr = device_msg_bytes.data_ptr() if hasattr(device_msg_bytes, "data_ptr") else int(device_msg_bytes)
    _check(_lib.bcast_exec_traced(_ptr_array(rank_bufs, "rank_bufs"), plan.handle, _stream_ptr(stream), mode,
                                  ctypes.c_void_p(ptr)), "bcast_exec_traced")


def bcast_exec_host(rank_bufs, plan: Plan, stream, mode: int, host_message, host_out=None) -> None:
    """``host_message``: host pointer (int), numpy array or CPU tensor with the message;
    ``host_out``: None or P entries, each None or a host pointer / array / CPU tensor to fill."""
    P = bcast_plan_num_ranks(plan)
    if len(rank_bufs) != P or (host_out is not None and len(host_out) != P):
        raise BcastError(BCAST_ERR_INVAL, "bcast_exec_host (array length != P)")

    def host_ptr(x):
        if x is None:
            return None
        if isinstance(x, np.ndarray):
            return x.ctypes.data
        if hasattr(x, "data_ptr"):
            return x.data_ptr()
        return int(x)
    outs = None if host_out is None else (ctypes.c_void_p * P)(*[host_ptr(x) for x in host_out])
    _check(_lib.bcast_exec_host(_ptr_array(rank_bufs, "rank_bufs"), plan.handle, _stream_ptr(stream), mode,
                                ctypes.c_void_p(host_ptr(host_message)), outs), "bcast_exec_host")


def bcast_exec_static(rank_bufs, plan: Plan, stream=None) -> None:
    """The broadcast for callers that must not allocate device memory (memory handed to a pool,
    fixed budgets, no tolerance for cudaMalloc's device-wide synchronisation): same arguments as
    :func:`bcast_exec`; the kernel's tables go into a fixed array inside the library instead of
    memory from cudaMalloc.  Raises ``BcastError`` with ``BCAST_ERR_CAPACITY`` when the plan's
    tables exceed ``BCAST_STATIC_SCRATCH_BYTES``.  Calls share that array: do not let two of them
    overlap on the GPU."""
    if len(rank_bufs) != bcast_plan_num_ranks(plan):
        raise BcastError(BCAST_ERR_INVAL, "bcast_exec_static (len(rank_bufs) != P)")
    _check(_lib.bcast_exec_static(_ptr_array(rank_bufs, "rank_bufs"), plan.handle, _stream_ptr(stream)),
           "bcast_exec_static")


def bcast_exec_status(plan: Plan) -> None:
    """After a stream synchronisation: raises ``BcastError`` (``BCAST_ERR_TIMEOUT``) if a kernel of
    this plan gave up on one of its bounded waits; returns None otherwise."""
    _check(_lib.bcast_exec_status(plan.handle), "bcast_exec_status")


def bcast_exec_num_launches(plan: Plan, mode: int = BCAST_EXEC_AUTO) -> int:
    return _lib.bcast_exec_num_launches(plan.handle, mode)


def bcast_strerror(code: int) -> str:
    return _lib.bcast_strerror(code).decode()


def bcast_last_cuda_error() -> int:
    return _lib.bcast_last_cuda_error()


# ---- the ranks of a plan spread over several GPUs
class Shard:
    """Owner of a ``bcast_shard_t*``; keeps its plan alive."""

    def __init__(self, handle: int, plan: Plan):
        self._h = ctypes.c_void_p(handle)
        self.plan = plan

    @property
    def handle(self) -> ctypes.c_void_p:
        if not self._h:
            raise ValueError("partition already freed")
        return self._h

    def free(self) -> None:
        if self._h:
            _lib.bcast_shard_free(self._h)
            self._h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def bcast_shard_create(plan: Plan, num_gpus: int, rank_gpu=None) -> Shard:
    arr = None
    if rank_gpu is not None:
        if len(rank_gpu) != bcast_plan_num_ranks(plan):
            raise BcastError(BCAST_ERR_INVAL, "bcast_shard_create (len(rank_gpu) != P)")
        arr = (ctypes.c_int32 * len(rank_gpu))(*[int(g) for g in rank_gpu])
    out = ctypes.c_void_p(None)
    _check(_lib.bcast_shard_create(plan.handle, num_gpus, arr, ctypes.byref(out)), "bcast_shard_create")
    return Shard(out.value, plan)


def bcast_shard_free(shard: Shard) -> None:
    shard.free()


def bcast_shard_num_gpus(shard: Shard) -> int: return _lib.bcast_shard_num_gpus(shard.handle)
def bcast_shard_num_phases(shard: Shard) -> int: return _lib.bcast_shard_num_phases(shard.handle)
def bcast_shard_crossing_bytes(shard: Shard) -> int: return _lib.bcast_shard_crossing_bytes(shard.handle)
def bcast_shard_crossing_msgs(shard: Shard) -> int: return _lib.bcast_shard_crossing_msgs(shard.handle)


def bcast_shard_rank_gpu(shard: Shard) -> np.ndarray:
    return _view(_lib.bcast_shard_rank_gpu(shard.handle), bcast_plan_num_ranks(shard.plan), np.int32)


def bcast_shard_msg_gpu(shard: Shard) -> np.ndarray:
    return _view(_lib.bcast_shard_msg_gpu(shard.handle), bcast_plan_num_xfers(shard.plan), np.int32)


def bcast_shard_msg_phase(shard: Shard, last: bool = False) -> np.ndarray:
    return _view(_lib.bcast_shard_msg_phase(shard.handle, int(last)), bcast_plan_num_xfers(shard.plan), np.int32)


def bcast_shard_hops(shard: Shard, phase: int, gpu: int, chunk: int) -> np.ndarray:
    n = _lib.bcast_shard_hops(shard.handle, phase, gpu, chunk, None, 0)
    if n < 0:
        raise BcastError(int(n), "bcast_shard_hops")
    out = np.zeros(int(n), dtype=np.int64)
    if n:
        got = _lib.bcast_shard_hops(shard.handle, phase, gpu, chunk, out.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), int(n))
        assert got == n
    return out


def _counter_ptr(device_msg_bytes) -> ctypes.c_void_p:
    if device_msg_bytes is None:
        return ctypes.c_void_p(None)
    return ctypes.c_void_p(device_msg_bytes.data_ptr() if hasattr(device_msg_bytes, "data_ptr") else int(device_msg_bytes))


def bcast_shard_exec(shard: Shard, rank_bufs, gpu_device, streams, device_msg_bytes=None) -> None:
    """``gpu_device``: CUDA device ordinal per GPU of the partition; ``streams``: one stream per GPU
    (torch streams or raw handles)."""
    G = bcast_shard_num_gpus(shard)
    if len(rank_bufs) != bcast_plan_num_ranks(shard.plan) or len(gpu_device) != G or len(streams) != G:
        raise BcastError(BCAST_ERR_INVAL, "bcast_shard_exec (array lengths)")
    devs = (ctypes.c_int * G)(*[int(d) for d in gpu_device])
    sts = (ctypes.c_void_p * G)(*[_stream_ptr(s).value for s in streams])
    _check(_lib.bcast_shard_exec(shard.handle, _ptr_array(rank_bufs, "rank_bufs"), devs, sts, _counter_ptr(device_msg_bytes)),
           "bcast_shard_exec")


def bcast_shard_exec_phase(shard: Shard, rank_bufs, phase: int, gpu: int, stream=None, device_msg_bytes=None) -> None:
    if len(rank_bufs) != bcast_plan_num_ranks(shard.plan):
        raise BcastError(BCAST_ERR_INVAL, "bcast_shard_exec_phase (len(rank_bufs) != P)")
    _check(_lib.bcast_shard_exec_phase(shard.handle, _ptr_array(rank_bufs, "rank_bufs"), phase, gpu, _stream_ptr(stream),
                                       _counter_ptr(device_msg_bytes)), "bcast_shard_exec_phase")

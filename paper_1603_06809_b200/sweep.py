"""Time the native and the tuned broadcast over a set of workloads on one GPU and print a table.

    python -m paper_1603_06809_b200.sweep [--set config5|paper|configs] [--mode auto|walk|walk_plan_order|walk_bulk|steps|graph]
                                           [--iters N] [--json]

For every workload: median time of the tuned and of the native variant (and, where P is a power of
two, of the scatter + recursive-doubling variant) (CUDA events around each
execution, after warm-up), the effective broadcast rate P*nbytes/t and its fraction of the measured
plain-copy rate (P*nbytes is what a broadcast cannot avoid moving through DRAM), the L2-level rate
2*sum(len)/t, and the tuned-over-native speed-up.  After timing, every rank buffer is compared with
the root's message on the device.  Uses only the CUDA library: no CPU path is involved.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics

import torch

from . import bcast as B
from . import workloads as W

MODES = {"walk": B.BCAST_EXEC_WALK, "walk_plan_order": B.BCAST_EXEC_WALK_PLAN_ORDER,
         "walk_bulk": B.BCAST_EXEC_WALK_BULK, "auto": B.BCAST_EXEC_AUTO,
         "steps": B.BCAST_EXEC_STEPS, "graph": B.BCAST_EXEC_GRAPH}


def time_workload(wl: W.Workload, variant: int, mode: int, iters: int, warmup: int = 5, device: str = "cuda:0"):
    """Median milliseconds of one broadcast, and the bytes its plan moves."""
    stride = (wl.nbytes + 511) // 256 * 256
    bufs = torch.empty((wl.P, stride), dtype=torch.uint8, device=device)
    for k in range(wl.P):
        bufs[k].fill_(W.poison_byte(k))
    msg = torch.from_numpy(W.message_bytes(wl.seed, wl.nbytes)).to(device)
    bufs[wl.root, : wl.nbytes].copy_(msg)
    ptrs = [bufs[k].data_ptr() for k in range(wl.P)]
    plan = B.bcast_plan(wl.P, wl.root, wl.nbytes, variant)
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        B.bcast_exec_mode(ptrs, plan, stream, mode)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    torch.cuda.synchronize()
    ev[0].record(stream)
    for i in range(iters):
        B.bcast_exec_mode(ptrs, plan, stream, mode)
        ev[i + 1].record(stream)
    torch.cuda.synchronize()
    ms = statistics.median(ev[i].elapsed_time(ev[i + 1]) for i in range(iters))
    if not all(torch.equal(bufs[k, : wl.nbytes], msg) for k in range(wl.P)):
        raise RuntimeError(f"{wl.name}: a rank buffer differs from the root's message")
    return ms, B.bcast_plan_total_bytes(plan)


def copy_rate_gbs() -> float:
    """The measured plain-copy rate of this machine's GPUs (MEASURED_PEAKS.json at the repository root),
    else the nominal 8000 GB/s: the denominator of the roofline fraction."""
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"])
    except Exception:
        return 8000.0


def run(workloads, mode: int, iters: int):
    peak = copy_rate_gbs()
    rows = []
    for wl in workloads:
        it = iters if wl.total_bytes < (1 << 30) else max(5, iters // 5)
        t_ms, t_bytes = time_workload(wl, B.BCAST_TUNED, mode, it)
        n_ms, n_bytes = time_workload(wl, B.BCAST_NATIVE, mode, it)
        d_ms = None
        if wl.P & (wl.P - 1) == 0:                       # recursive doubling needs a power of two
            d_ms, _ = time_workload(wl, B.BCAST_DOUBLING, mode, it)
        rows.append({
            "workload": wl.name, "P": wl.P, "nbytes": wl.nbytes,
            "doubling_us": None if d_ms is None else round(d_ms * 1e3, 2),
            "tuned_us": round(t_ms * 1e3, 2), "native_us": round(n_ms * 1e3, 2),
            "tuned_effective_GBps": round(wl.P * wl.nbytes / t_ms / 1e6, 1),
            # DRAM floor of a broadcast (message read once, every other buffer written once = P*nbytes) over the copy rate
            "tuned_roofline_frac": round(wl.P * wl.nbytes / t_ms / 1e6 / peak, 4),
            "native_roofline_frac": round(wl.P * wl.nbytes / n_ms / 1e6 / peak, 4),
            "tuned_algorithmic_GBps": round(2 * t_bytes / t_ms / 1e6, 1),
            "native_algorithmic_GBps": round(2 * n_bytes / n_ms / 1e6, 1),
            "bytes_native_over_tuned": round(n_bytes / t_bytes, 4) if t_bytes else None,
            "speedup_tuned_over_native": round(n_ms / t_ms, 4),
        })
        torch.cuda.empty_cache()
    return rows


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--set", default="paper", choices=["config5", "paper", "configs"])
    ap.add_argument("--mode", default="auto", choices=sorted(MODES))
    ap.add_argument("--iters", type=int, default=50)
    ap.add_argument("--json", action="store_true", help="one JSON object per line instead of a table")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: there is no CPU fallback")
    wls = {"config5": W.sweep, "paper": W.paper_experiments,
           "configs": lambda: [W.CFG1, W.CFG2, W.CFG3, W.CFG4]}[args.set]()
    rows = run(wls, MODES[args.mode], args.iters)
    if args.json:
        for r in rows:
            print(json.dumps(r))
        return
    print(f"{'workload':28s} {'tuned us':>10s} {'native us':>10s} {'P*n/t GB/s':>11s} {'roofline':>8s} {'L2 GB/s':>10s} "
          f"{'bytes n/t':>9s} {'speed-up':>8s} {'doubling us':>11s}")
    for r in rows:
        print(f"{r['workload']:28s} {r['tuned_us']:10.2f} {r['native_us']:10.2f} {r['tuned_effective_GBps']:11.1f} "
              f"{r['tuned_roofline_frac']:8.3f} {r['tuned_algorithmic_GBps']:10.1f} {r['bytes_native_over_tuned']:9.4f} {r['speedup_tuned_over_native']:8.4f} "
              f"{'' if r['doubling_us'] is None else format(r['doubling_us'], '11.2f')}")


if __name__ == "__main__":
    main()

"""Scatter-ring-allgather broadcast (native and bandwidth-saving tuned ring) over P virtual ranks
in one GPU's memory: thin Python binding of the C-ABI library built from ``csrc/``.

``from paper_1603_06809_b200 import bcast`` loads the shared library; it raises if the library
has not been built (``python -m paper_1603_06809_b200.build``).  There is no CPU fallback.
"""
__all__ = ["bcast", "workloads", "build"]

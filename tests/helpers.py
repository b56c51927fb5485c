"""Helpers shared by the test files (no arithmetic of the CUDA path or of the oracle)."""
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def golden_path(name):
    return os.path.join(ROOT, "tests", "golden", name)


def golden_lines(name):
    with open(golden_path(name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]

"""Writes tests/golden/oracle_cfg1_rows.txt: a few output rows and lse values of the tiny
forward workload, computed by the CPU oracle alone (no CUDA code is imported or run).

Run from the repository root:  python tests/golden/make_golden.py
The file guards the oracle against silent drift; the oracle's correctness itself is pinned by
tests/test_oracle_pins.py, not by this file.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2508_20407_b200 import synth  # noqa: E402  (seeded inputs only)

ROWS = [(0, 0, 0), (0, 1, 17), (0, 2, 64), (0, 3, 127)]


def main():
    wl = synth.WORKLOADS["cfg1_tiny"]
    q, k, v = synth.forward_inputs(wl)
    out, lse = oracle.attn_forward(q, k, v, wl.causal_window)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_cfg1_rows.txt")
    with open(path, "w") as f:
        f.write("# oracle outputs for workload cfg1_tiny (B1 H4 d64 N1024 W128, causal window), written by make_golden.py\n")
        f.write("# b h i lse out[0..7]\n")
        for b, h, i in ROWS:
            vals = " ".join(f"{x:.17g}" for x in out[b, h, i, :8])
            f.write(f"{b} {h} {i} {lse[b, h, i]:.17g} {vals}\n")
    print("wrote", path)


if __name__ == "__main__":
    main()

"""Writes tests/golden/prune_small.txt from the CPU oracle alone.

Run from the repository root:  python tests/golden/make_golden.py
The file freezes the oracle's packed output for two tiny seeded tensors so that an
unintended change to its arithmetic, block numbering or packing is noticed.  Nothing
in it comes from the CUDA path.
"""
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parents[2]
sys.path.insert(0, str(ROOT))

import oracle  # noqa: E402
from paper_2203_10991_b200 import workloads  # noqa: E402


def main():
    lines = ["# oracle.prune on workloads.gradient((16, 16), dist, seed=0); prune seed 42",
             "# columns: dist n m axis joint | values (hex, row-major) | meta (hex, row-major)",
             "# joint: 0 = pair table of App. A.2, 1 = systematic sampling, 2 = approx-MVUE of Sec. 4.4 (2:4 only);",
             "# n m = 1 4 is MVUE 1:4 (one survivor beside a +0 in the 2:4 container)"]
    for dist, dtype in (("relu_normal", "f32"), ("student_t", "bf16")):
        g = workloads.gradient((16, 16), dist, seed=0, dtype=dtype)
        for (n, m, joint) in ((1, 2, 0), (2, 4, 0), (2, 4, 1), (2, 4, 2), (1, 4, 0)):
            for axis in (0, 1):
                v, mt = oracle.prune(g, n, m, axis=axis, seed=42, joint=joint)
                lines.append(f"{dist} {n} {m} {axis} {joint} | " + v.tobytes().hex() + " | " + mt.tobytes().hex())
    (Path(__file__).parent / "prune_small.txt").write_text("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()

"""The oracle still reproduces the packed output frozen under tests/golden/ (written by
tests/golden/make_golden.py from the oracle alone)."""
from pathlib import Path

import numpy as np

import oracle
from paper_2203_10991_b200 import workloads


def test_frozen_packed_output():
    rows = [l for l in (Path(__file__).parent / "golden" / "prune_small.txt").read_text().splitlines()
            if l and not l.startswith("#")]
    assert len(rows) == 20
    for row in rows:
        head, vhex, mhex = [s.strip() for s in row.split("|")]
        dist, n, m, axis, joint = head.split()
        g = workloads.gradient((16, 16), dist, seed=0, dtype="f32" if dist == "relu_normal" else "bf16")
        v, mt = oracle.prune(g, int(n), int(m), axis=int(axis), seed=42, joint=int(joint))
        assert v.tobytes().hex() == vhex and mt.tobytes().hex() == mhex

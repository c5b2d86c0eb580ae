"""Pins for the oracle's counter-based generator (Philox4x32-10, SC'11).

The C oracle is compared with (i) an independent big-integer restatement and
(ii) the generator header that ships with PyTorch, compiled here as a probe.
"""
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest

import oracle
from oracle import philox_py

TORCH_INCLUDE = None


def _torch_include():
    import torch
    return Path(torch.__file__).parent / "include"


def test_c_matches_bigint_restatement():
    rng = np.random.Generator(np.random.PCG64(11))
    for _ in range(20000):
        ctr = [int(x) for x in rng.integers(0, 2**32, 4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 2**32, 2, dtype=np.uint64)]
        assert oracle.philox4x32_10(ctr, key) == philox_py.philox4x32(ctr, key)
    # structured counters: zeros, all ones, single bits
    for ctr, key in [((0, 0, 0, 0), (0, 0)), ((2**32 - 1,) * 4, (2**32 - 1,) * 2)] + \
                    [((1 << b, 0, 0, 0), (0, 1 << b)) for b in range(32)]:
        assert oracle.philox4x32_10(ctr, key) == philox_py.philox4x32(ctr, key)


def test_c_matches_pytorch_header(tmp_path):
    probe = tmp_path / "probe"
    src = Path(__file__).parent / "helpers" / "philox_torch_probe.cpp"
    subprocess.run(["g++", "-O1", "-std=c++17", f"-I{_torch_include()}", str(src), "-o", str(probe)],
                   check=True)
    rng = np.random.Generator(np.random.PCG64(5))
    cases = [(0, 0), (1, 0), (0, 1), (2**64 - 1, 2**40 + 3)]
    cases += [(int(rng.integers(0, 2**63)) * 2 + int(rng.integers(0, 2)), int(rng.integers(0, 2**48)))
              for _ in range(500)]
    args = []
    for seed, call in cases:
        args += [str(seed), "0", str(call)]
    out = subprocess.run([str(probe), *args], check=True, capture_output=True, text=True).stdout
    rows = [tuple(int(x) for x in line.split()) for line in out.strip().splitlines()]
    assert len(rows) == len(cases)
    for (seed, call), row in zip(cases, rows):
        ctr = (call & 0xFFFFFFFF, call >> 32, 0, 0)
        key = (seed & 0xFFFFFFFF, seed >> 32)
        assert oracle.philox4x32_10(ctr, key) == row
        # and the per-block word: call number q >> 2, lane q & 3
        for lane in range(4):
            assert oracle.block_word(seed, 4 * call + lane) == row[lane]
            assert philox_py.block_word(seed, 4 * call + lane) == row[lane]


def test_fewer_rounds_differ():
    # guards the round count: 7 or 9 rounds must not reproduce the 10-round words
    for r in (7, 9, 11):
        assert philox_py.philox4x32((1, 2, 3, 4), (5, 6), rounds=r) != oracle.philox4x32_10((1, 2, 3, 4), (5, 6))


def test_uniform24_exact_and_in_range():
    assert oracle.uniform24(0) == 0.0
    assert oracle.uniform24(0xFF) == 0.0                       # low 8 bits are unused
    assert oracle.uniform24(0x100) == 2.0 ** -24
    assert oracle.uniform24(0xFFFFFFFF) == 1.0 - 2.0 ** -24    # never reaches 1
    assert oracle.uniform24(0x80000000) == 0.5


def test_uniformity_chi_square():
    words = np.array([oracle.block_word(123, q) for q in range(1 << 17)], dtype=np.uint64)
    u = (words >> 8).astype(np.float64) / 2**24
    bins = np.bincount((u * 64).astype(int), minlength=64)
    expected = len(u) / 64
    chi2 = ((bins - expected) ** 2 / expected).sum()
    assert chi2 < 120.0            # 63 dof: P(chi2 > 120) ~ 1e-5
    assert abs(u.mean() - 0.5) < 5 * (1 / 12 / len(u)) ** 0.5
    # lanes of one call and neighbouring calls are not trivially related
    assert len(set(int(w) for w in words[:4096])) > 4090

"""The C-ABI library builds, loads and exports what include/mvue.h declares; host-side
argument checks answer without a GPU."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def L():
    from paper_2203_10991_b200 import build, binding
    build.build()
    return binding.lib()


def declared_symbols():
    names = []
    for header in sorted((ROOT / "include").glob("*.h")):
        names += re.findall(r"MVUE_API\s+[\w\s\*]+?\b(mvue_\w+)\s*\(", header.read_text())
    return names


def test_every_declared_symbol_is_exported(L):
    names = declared_symbols()
    assert len(names) >= 6 and "mvue_prune" in names
    for name in names:
        assert hasattr(L, name), f"{name} declared in include/ but not exported"
    from paper_2203_10991_b200 import binding
    assert set(binding.EXPORTS) == set(names)


def test_version_and_status_strings(L):
    assert L.mvue_version() >= 100
    seen = set()
    for code in range(0, -11, -1):
        s = L.mvue_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 11
    assert L.mvue_status_string(-99).decode() == "unknown status"


def test_packed_sizes_and_host_side_checks(L):
    from paper_2203_10991_b200 import binding
    assert binding.mvue_packed_sizes(512, 256, 1, 2, 0) == (256 * 256 * 2, 256 * 64)
    assert binding.mvue_packed_sizes(512, 256, 2, 4, 1) == (512 * 128 * 2, 512 * 32)
    assert binding.mvue_packed_sizes(512, 256, 1, 4, 1) == (512 * 128 * 2, 512 * 32)    # 1:4 sits in the 2:4 container
    for n, m in [(3, 4), (4, 8), (2, 2), (0, 0)]:
        with pytest.raises(binding.MvueError) as e:
            binding.mvue_packed_sizes(512, 256, n, m, 0)
        assert e.value.status == -2
    for rows, cols, axis in [(500, 256, 0), (512, 250, 1), (512, 252, 0), (0, 16, 1), (16, 16, 2)]:
        with pytest.raises(binding.MvueError) as e:
            binding.mvue_packed_sizes(rows, cols, 2, 4, axis)
        assert e.value.status == -3
    with pytest.raises(binding.MvueError) as e:
        binding.mvue_packed_sizes(512, 256, 2, 4, 0, layout=7)
    assert e.value.status == -6
    # checks that come before any CUDA call: NULL pointers, dtype, shard bounds, alignment
    assert L.mvue_prune(None, 1, 16, 16, 16, 2, 4, 1, 0, 16, 0, None, None, 0, None) == -1
    fake = ctypes.c_void_p(4096)
    assert L.mvue_prune(fake, 5, 16, 16, 16, 2, 4, 1, 0, 16, 0, fake, fake, 0, None) == -5
    assert L.mvue_prune(fake, 1, 16, 16, 8, 2, 4, 1, 0, 16, 0, fake, fake, 0, None) == -3      # ld < cols
    assert L.mvue_prune(fake, 1, 16, 16, 16, 2, 4, 1, 0, 32, 32, fake, fake, 0, None) == -3    # shard outside K
    assert L.mvue_prune(ctypes.c_void_p(4100), 1, 16, 16, 16, 2, 4, 1, 0, 16, 0, fake, fake, 0, None) == -4
    assert L.mvue_prune(fake, 1, 16, 16, 20, 2, 4, 1, 0, 16, 0, fake, fake, 0, None) == -4     # ld * 2 % 16
    assert L.mvue_unpack(None, fake, 0, 16, 16, fake, None) == -1
    # the allocation-free update product checks its arguments like the regular one, before any CUDA call
    na = L.mvue_sparse_update_gemm_noalloc
    assert na(None, fake, 1, 256, 512, fake, 256, 256, fake, 0, 256, 0, None, None) == -1
    assert na(fake, fake, 0, 256, 512, fake, 256, 256, fake, 0, 256, 0, None, None) == -6          # canonical layout
    assert na(fake, fake, 1, 256, 500, fake, 256, 256, fake, 0, 256, 0, None, None) == -3          # T % 128
    assert na(fake, fake, 1, 256, 512, ctypes.c_void_p(4100), 256, 256, fake, 0, 256, 0, None, None) == -4
    assert na(fake, fake, 1, 256, 512, fake, 256, 256, fake, 1, 256, 1, None, None) == -5          # bf16 += is not offered
    # the bounded-wait self-test: a status word is required, the poll count is bounded
    assert L.mvue_selftest_wait_timeout(100, None, None) == -1
    assert L.mvue_selftest_wait_timeout(0, fake, None) == -3
    assert L.mvue_selftest_wait_timeout(1 << 20, fake, None) == -3


def test_no_silent_cpu_path(L):
    """Without a CUDA device the library reports an error instead of computing anything."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    fake = ctypes.c_void_p(4096)
    assert L.mvue_prune(fake, 1, 16, 16, 16, 2, 4, 1, 0, 16, 0, fake, fake, 0, None) in (-8, -9)

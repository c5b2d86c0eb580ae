"""Two CPU ranks (gloo): token shards pruned with the global block numbering and summed by an all-reduce
reproduce the unsharded update product.  Exercises the host-side shard arithmetic and the exchange step of
the data-parallel path; the per-shard arithmetic here is the oracle's (no GPU in this test)."""
import os
import socket
import sys
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))

from paper_2203_10991_b200 import sharding, workloads  # noqa: E402

T, OUT, INP, SEED = 1024 + 128, 24, 16, 77


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = workloads.gradient((T, OUT), "student_t", seed=1, dtype="bf16")
    h = workloads.normal_bf16((T, INP), seed=2)
    off, n = sharding.token_shard(T, world, rank)
    v, m = oracle.prune(np.ascontiguousarray(g[off:off + n]), 2, 4, axis=0, seed=SEED, k_total=T, k_offset=off)
    part = torch.from_numpy(oracle.gemm(oracle.unpack(v, m), h[off:off + n]))
    dist.all_reduce(part)
    # the same shard arguments through the library's own argument checks (no GPU here: a valid call stops at the
    # device lookup, -8 or -9; a shard that sticks out of the global K, or is off the 16-row grid, is refused as a
    # shape error before that)
    import ctypes
    from paper_2203_10991_b200 import binding
    L = binding.lib()
    fake = ctypes.c_void_p(1 << 20)
    codes = (L.mvue_prune_joint(fake, 1, n, OUT, OUT, 2, 4, 0, SEED, T, off, fake, fake, 1, 1, None),
             L.mvue_prune_joint(fake, 1, n, OUT, OUT, 2, 4, 0, SEED, T, T - n + 128, fake, fake, 1, 1, None),
             L.mvue_prune_joint(fake, 1, n, OUT, OUT, 2, 4, 0, SEED, T, off + 8, fake, fake, 1, 1, None))
    if rank == 0:
        q.put((part.numpy(), off, n, codes))
    dist.destroy_process_group()


def test_two_rank_token_shards_sum_to_the_unsharded_update():
    import oracle
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got, off0, n0, codes = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    g = workloads.gradient((T, OUT), "student_t", seed=1, dtype="bf16")
    h = workloads.normal_bf16((T, INP), seed=2)
    v, m = oracle.prune(g, 2, 4, axis=0, seed=SEED)
    want = oracle.gemm(oracle.unpack(v, m), h)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-15)
    assert (off0, n0) == (0, 640)                      # 9 granules over 2 ranks: 5 + 4
    has_gpu = torch.cuda.is_available()
    assert codes[0] in ((0,) if has_gpu else (-8, -9)) or has_gpu
    assert codes[1] == -3 and codes[2] == -3


def test_token_shard_properties():
    for total, world in [(128, 1), (1152, 2), (200704, 8), (16384, 3), (256, 4)]:
        spans = [sharding.token_shard(total, world, r) for r in range(world)]
        assert spans[0][0] == 0 and sum(n for _, n in spans) == total
        for (o1, n1), (o2, _) in zip(spans, spans[1:]):
            assert o1 + n1 == o2
        assert all(o % 128 == 0 and n % 128 == 0 for o, n in spans)
        assert max(n for _, n in spans) - min(n for _, n in spans) <= 128
    with pytest.raises(ValueError):
        sharding.token_shard(100, 2, 0)
    with pytest.raises(ValueError):
        sharding.token_shard(256, 2, 2)

"""Approx-4:8 prune (prune only): the CUDA kernel against the CPU oracle, masks and packed survivors bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_10991_b200 import binding, workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)
    return torch.from_numpy(a).to(DEV)


def gpu(g_np, axis, seed, **kw):
    values, mask = binding.mvue_prune_4of8(to_dev(g_np), axis, seed, **kw)
    torch.cuda.synchronize()
    return values.view(torch.int16).cpu().numpy().view(np.uint16), mask.cpu().numpy()


@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", [(8, 8), (48, 80), (520, 264), (1024, 512)])
@pytest.mark.parametrize("dist,dtype", [("relu_normal", "f32"), ("relu_lognormal", "bf16"), ("student_t", "bf16"),
                                        ("student_t", "f32")])
def test_bit_parity(axis, shape, dist, dtype):
    g = workloads.gradient(shape, dist, seed=shape[0] + shape[1], dtype=dtype)
    seed = 0x9E3779B97F4A7C15 ^ shape[1]
    v_gpu, m_gpu = gpu(g, axis, seed)
    v_ref, m_ref = oracle.prune_4of8(g, axis, seed, threads=oracle.host_threads())
    assert np.array_equal(m_gpu, m_ref), np.flatnonzero(m_gpu.ravel() != m_ref.ravel())[:4]
    bad = np.flatnonzero(v_gpu.ravel() != v_ref.ravel())
    assert bad.size == 0, f"{bad.size} survivors differ, first at {bad[:4]}"
    assert all(bin(int(b)).count("1") == 4 for b in m_gpu.ravel()[:4096])


def test_zero_blocks_ties_and_k_shards():
    rng = np.random.Generator(np.random.PCG64(5))
    pool = np.array([0.0, -0.0, 1.0, -1.0, 2.0, 3.0, 0.5, 1e-3, 1e3, 1.5, 7.0, -0.25], dtype=np.float32)
    g = pool[rng.integers(0, len(pool), size=(64, 128))]
    g[0, :16] = [0, 2, 0, 0, -3, 0, 0, 0, 1, 0, 2, 0, 3, 0, 4, 0]
    g[1, :16] = [0] * 8 + [1] * 8
    for dtype in ("f32", "bf16"):
        gg = np.ascontiguousarray(workloads.to_bf16_bits(g) if dtype == "bf16" else g)
        for axis in (0, 1):
            v_gpu, m_gpu = gpu(gg, axis, 77)
            v_ref, m_ref = oracle.prune_4of8(gg, axis, 77)
            assert np.array_equal(m_gpu, m_ref) and np.array_equal(v_gpu, v_ref), (dtype, axis)
    K = 128
    v_all, m_all = oracle.prune_4of8(g, 1, 31)
    for lo, hi in [(0, 48), (48, K)]:
        v, mk = gpu(np.ascontiguousarray(g[:, lo:hi]), 1, 31, k_total=K, k_offset=lo)
        assert np.array_equal(v, v_all[:, lo // 2:hi // 2]) and np.array_equal(mk, m_all[:, lo // 8:hi // 8])


def test_bad_arguments():
    g = to_dev(workloads.gradient((64, 64), "student_t", seed=1, dtype="bf16"))
    with pytest.raises(binding.MvueError) as e:
        binding.mvue_prune_4of8(g[:, :36], 1, 0)               # K = 36 is not a multiple of 8
    assert e.value.status == -3
    with pytest.raises(binding.MvueError) as e:
        binding.mvue_prune_4of8(g, 2, 0)
    assert e.value.status == -3

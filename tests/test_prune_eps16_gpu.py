"""MVUE_OPT_EPS16 (sixteen random bits per block, one generator call per eight blocks): bit parity of every CUDA prune
kernel with the CPU oracle, alone and together with stochastic rounding, and unbiasedness over seeds."""
import numpy as np
import pytest
import torch

import oracle
from oracle import theory
from paper_2203_10991_b200 import binding, workloads
from tests.helpers import layouts

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
E16, SR = binding.MVUE_OPT_EPS16, binding.MVUE_OPT_STOCHASTIC_ROUNDING
ESTIMATORS = [(1, 2, 0), (2, 4, 0), (2, 4, 1), (2, 4, 2), (1, 4, 0)]


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)
    return torch.from_numpy(a).to(DEV)


def gpu(g_np, n, m, joint, axis, seed, options=E16, **kw):
    values, meta = binding.mvue_prune(to_dev(g_np), n, m, axis, seed, joint=joint, options=options, **kw)
    torch.cuda.synchronize()
    return values.view(torch.int16).cpu().numpy().view(np.uint16), meta.cpu().numpy()


SHAPES = [(48, 80), (528, 264), (256, 192), (1152, 320), (176, 1536), (512, 256), (384, 64)]        # ragged; whole 128 x 64 tiles (a kernel of its own down the rows)


@pytest.mark.parametrize("n,m,joint", ESTIMATORS)
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dist,dtype", [("relu_normal", "f32"), ("relu_lognormal", "bf16"), ("student_t", "bf16")])
@pytest.mark.parametrize("sr", [False, True])
def test_bit_parity(n, m, joint, axis, shape, dist, dtype, sr):
    rows, cols = shape
    if axis == 1:
        cols = (cols + 15) // 16 * 16
    else:
        rows, cols = (rows + 15) // 16 * 16, (cols + 7) // 8 * 8
    g = workloads.gradient((rows, cols), dist, seed=rows + cols, dtype=dtype)
    seed = 0xD1B54A32D192ED03 ^ rows
    v_gpu, m_gpu = gpu(g, n, m, joint, axis, seed, options=E16 | (SR if sr else 0))
    v_ref, m_ref = oracle.prune(g, n, m, axis=axis, seed=seed, joint=joint, eps16=True, stochastic_rounding=sr,
                                threads=oracle.host_threads())
    bad_m = np.flatnonzero(m_gpu.ravel() != m_ref.ravel())
    assert bad_m.size == 0, f"{bad_m.size} metadata bytes differ, first at {bad_m[:4]}"
    bad_v = np.flatnonzero(v_gpu.ravel() != v_ref.ravel())
    assert bad_v.size == 0, f"{bad_v.size} packed values differ, first at {bad_v[:4]}"
    if not sr:                                                   # another stream of bits than the 32-bit one
        _, m_32 = oracle.prune(g, n, m, axis=axis, seed=seed, joint=joint)
        assert not np.array_equal(m_32, m_ref)


@pytest.mark.parametrize("n,m,joint", ESTIMATORS)
@pytest.mark.parametrize("axis", [0, 1])
def test_tensor_core_order_and_k_shards(n, m, joint, axis):
    g = workloads.gradient((256, 256), "student_t", seed=8, dtype="bf16")
    K = 256
    v_all, m_all = oracle.prune(g, n, m, axis=axis, seed=41, joint=joint, eps16=True)
    values, meta = binding.mvue_prune(to_dev(g), n, m, axis, 41, joint=joint, options=E16, layout=binding.MVUE_LAYOUT_TC)
    torch.cuda.synchronize()
    assert np.array_equal(values.view(torch.int16).cpu().numpy().view(np.uint16), v_all)
    assert np.array_equal(meta.cpu().numpy().reshape(-1), layouts.canonical_to_tc(m_all))
    # shards on the 128 grid, and one whose first unit is odd (the two units of a lane then sit in different calls)
    for lo, hi in [(0, 128), (128, K), (16, 144)]:
        part = np.ascontiguousarray(g[:, lo:hi] if axis == 1 else g[lo:hi])
        v, mt = gpu(part, n, m, joint, axis, 41, k_total=K, k_offset=lo)
        assert np.array_equal(v, v_all[:, lo // 2:hi // 2]) and np.array_equal(mt, m_all[:, lo // 8:hi // 8]), (lo, hi)


def test_edge_values():
    rng = np.random.Generator(np.random.PCG64(29))
    pool = np.array([0.0, -0.0, 1.0, -1.0, 2.0, 3.0, 5.0, 6.0, 0.5, 1e-3, 1e3, 2.0**-126, 2.0**-133, -2.0**-130,
                     2.0**100, -2.0**120, 1.5, 1.75, 3.0e-39], dtype=np.float32)
    g = pool[rng.integers(0, len(pool), size=(256, 128))]
    for dtype in ("f32", "bf16"):
        gg = np.ascontiguousarray(workloads.to_bf16_bits(g) if dtype == "bf16" else g)
        for n, m, joint in ESTIMATORS:
            for axis in (0, 1):
                v_gpu, m_gpu = gpu(gg, n, m, joint, axis, 2**63 + 9)
                v_ref, m_ref = oracle.prune(gg, n, m, axis=axis, seed=2**63 + 9, joint=joint, eps16=True)
                assert np.array_equal(m_gpu, m_ref) and np.array_equal(v_gpu, v_ref), (dtype, n, m, joint, axis)


def test_unbiased_over_10k_seeds():
    cfg = workloads.CONFIGS["linear_small"]
    g = np.ascontiguousarray(workloads.gradient((cfg["T"], cfg["out"]), cfg["g_dist"], cfg["seed"], dtype="f32")[:16, :16])
    g_dev = to_dev(g)
    n_seeds = 10000
    acc = torch.zeros((16, 16), dtype=torch.float64, device=DEV)
    values = torch.empty((16, 8), dtype=torch.bfloat16, device=DEV)
    meta = torch.empty((16, 2), dtype=torch.uint8, device=DEV)
    for seed in range(n_seeds):
        binding.mvue_prune(g_dev, 2, 4, 0, seed, values=values, meta=meta, joint=binding.MVUE_JOINT_SYSTEMATIC, options=E16)
        acc += binding.mvue_unpack(values, meta).double()
    mean = (acc / n_seeds).cpu().numpy()
    A = g.T.astype(np.float64)
    for r in range(16):
        for j in range(4):
            blk = A[r, 4 * j:4 * j + 4]
            p = (blk != 0).astype(np.float64) if np.count_nonzero(blk) < 2 else theory.marginals24(blk)
            for e in range(4):
                a = blk[e]
                if a == 0:
                    assert mean[r, 4 * j + e] == 0
                    continue
                sd = np.sqrt(a * a * max(1 / p[e] - 1, 0.0) / n_seeds)
                assert abs(mean[r, 4 * j + e] - a) <= 6 * sd + 2.0 ** -8 * abs(a), (r, j, e)

"""Stochastic rounding of the survivors (mvue_prune_opts, MVUE_OPT_STOCHASTIC_ROUNDING): bit parity of the CUDA
kernels with the CPU oracle for every estimator, axis, input type and layout, and the property the option exists
for -- the mean of the stored values over seeds converges on the gradient with no 2^-9 storage bias left."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_10991_b200 import binding, workloads
from tests.helpers import layouts

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SR = binding.MVUE_OPT_STOCHASTIC_ROUNDING
ESTIMATORS = [(1, 2, 0), (2, 4, 0), (2, 4, 1), (2, 4, 2), (1, 4, 0)]          # (n, m, joint)


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)
    return torch.from_numpy(a).to(DEV)


def gpu(g_np, n, m, joint, axis, seed, **kw):
    values, meta = binding.mvue_prune(to_dev(g_np), n, m, axis, seed, joint=joint, options=SR, **kw)
    torch.cuda.synchronize()
    return values.view(torch.int16).cpu().numpy().view(np.uint16), meta.cpu().numpy()


# ragged shapes (general kernels) and shapes of whole 128 x 64 tiles (the bf16 kernel of its own down the rows)
SHAPES = [(48, 80), (528, 264), (256, 192), (1152, 320), (176, 1536), (512, 256), (384, 64)]


@pytest.mark.parametrize("n,m,joint", ESTIMATORS)
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dist,dtype", [("relu_normal", "f32"), ("relu_lognormal", "bf16"), ("student_t", "bf16")])
def test_bit_parity_with_stochastic_rounding(n, m, joint, axis, shape, dist, dtype):
    rows, cols = shape
    if axis == 1:
        cols = (cols + 15) // 16 * 16
    else:
        rows, cols = (rows + 15) // 16 * 16, (cols + 7) // 8 * 8
    g = workloads.gradient((rows, cols), dist, seed=rows + cols, dtype=dtype)
    seed = 0x9E3779B97F4A7C15 ^ cols
    v_gpu, m_gpu = gpu(g, n, m, joint, axis, seed)
    v_ref, m_ref = oracle.prune(g, n, m, axis=axis, seed=seed, joint=joint, stochastic_rounding=True,
                                threads=oracle.host_threads())
    assert np.array_equal(m_gpu, m_ref)
    bad = np.flatnonzero(v_gpu.ravel() != v_ref.ravel())
    assert bad.size == 0, f"{bad.size} packed values differ, first at {bad[:4]}"
    # and the option did something: against round-to-nearest some survivors moved by one bf16 step, none by more
    v_rn, m_rn = oracle.prune(g, n, m, axis=axis, seed=seed, joint=joint, threads=oracle.host_threads())
    assert np.array_equal(m_rn, m_ref)
    step = v_gpu.astype(np.int32) - v_rn.astype(np.int32)
    assert np.abs(step).max() <= 1
    if dtype == "f32" or (n, m) != (2, 4) or joint == 2:
        assert np.count_nonzero(step) > 0


@pytest.mark.parametrize("n,m,joint", ESTIMATORS)
@pytest.mark.parametrize("axis", [0, 1])
def test_tensor_core_order_and_k_shards(n, m, joint, axis):
    g = workloads.gradient((256, 256), "student_t", seed=8, dtype="bf16")
    K = 256
    v_all, m_all = oracle.prune(g, n, m, axis=axis, seed=41, joint=joint, stochastic_rounding=True)
    values, meta = binding.mvue_prune(to_dev(g), n, m, axis, 41, joint=joint, options=SR, layout=binding.MVUE_LAYOUT_TC)
    torch.cuda.synchronize()
    assert np.array_equal(values.view(torch.int16).cpu().numpy().view(np.uint16), v_all)
    assert np.array_equal(meta.cpu().numpy().reshape(-1), layouts.canonical_to_tc(m_all))
    for lo, hi in [(0, 128), (128, K)]:
        part = np.ascontiguousarray(g[:, lo:hi] if axis == 1 else g[lo:hi])
        v, mt = gpu(part, n, m, joint, axis, 41, k_total=K, k_offset=lo)
        assert np.array_equal(v, v_all[:, lo // 2:hi // 2]) and np.array_equal(mt, m_all[:, lo // 8:hi // 8])


def test_edge_values_with_stochastic_rounding():
    rng = np.random.Generator(np.random.PCG64(23))
    pool = np.array([0.0, -0.0, 1.0, -1.0, 2.0, 3.0, 5.0, 6.0, 0.5, 1e-3, 1e3, 2.0**-126, 2.0**-133, -2.0**-130,
                     2.0**100, -2.0**120, 1.5, 1.75, 3.0e-39, 1.0 + 2.0**-20, -(2.0 - 2.0**-23)], dtype=np.float32)
    g = pool[rng.integers(0, len(pool), size=(256, 128))]
    for dtype in ("f32", "bf16"):
        gg = workloads.to_bf16_bits(g) if dtype == "bf16" else g
        for n, m, joint in ESTIMATORS:
            for axis in (0, 1):
                v_gpu, m_gpu = gpu(np.ascontiguousarray(gg), n, m, joint, axis, 2**63 + 5)
                v_ref, m_ref = oracle.prune(np.ascontiguousarray(gg), n, m, axis=axis, seed=2**63 + 5, joint=joint,
                                            stochastic_rounding=True)
                assert np.array_equal(m_gpu, m_ref) and np.array_equal(v_gpu, v_ref), (dtype, n, m, joint, axis)


def test_unknown_option_bits_are_refused():
    g = to_dev(workloads.gradient((64, 64), "student_t", seed=1, dtype="bf16"))
    with pytest.raises(binding.MvueError) as e:
        binding.mvue_prune(g, 2, 4, 1, 0, options=0x80)
    assert e.value.status == -12


@pytest.mark.parametrize("n,m,joint", [(2, 4, 1), (2, 4, 0), (1, 2, 0)])
def test_mean_over_seeds_has_no_storage_bias(n, m, joint):
    # blocks built so that every rescaled survivor sits a quarter of the way between two bf16 numbers: round-to-nearest
    # then stores the lower neighbour every time (a relative bias of 2^-10 on the block sum, 40 standard errors here),
    # stochastic rounding leaves the mean on the gradient
    if m == 4:
        block = [1.0, 1.0, 1.0, 1.0 + 2.0**-6]                 # sum / 2 = 2 + 2^-7
    else:
        block = [1.0, 1.0 + 2.0**-7, 1.0, 1.0 + 2.0**-7]       # pair sums 2 + 2^-7
    g = np.tile(np.array(block, dtype=np.float32), (16, 16))   # [16 x 64], blocks along the rows of g (axis 1)
    g_dev = to_dev(g)
    n_seeds = 4000
    acc = {0: torch.zeros_like(g_dev, dtype=torch.float64), SR: torch.zeros_like(g_dev, dtype=torch.float64)}
    values = torch.empty((16, 32), dtype=torch.bfloat16, device=DEV)
    meta = torch.empty((16, 8), dtype=torch.uint8, device=DEV)
    for seed in range(n_seeds):
        for opt in (0, SR):
            binding.mvue_prune(g_dev, n, m, 1, seed, values=values, meta=meta, joint=joint, options=opt)
            acc[opt] += binding.mvue_unpack(values, meta).double()
    total = float(g.astype(np.float64).sum())
    mean_rn, mean_sr = float(acc[0].sum()) / n_seeds, float(acc[SR].sum()) / n_seeds
    n_survivors = g.size // 2
    sd = np.sqrt(n_survivors * (2.0**-7 * np.sqrt(3) / 4) ** 2 / n_seeds)    # rounding noise: +-2^-7 steps w.p. 1/4, 3/4
    assert abs(mean_rn - total * 2.0 / (2.0 + 2.0**-7)) < 1e-6 * total
    assert abs(mean_sr - total) < 6 * sd
    assert abs(mean_rn - total) > 20 * sd

"""Parity of the CUDA prune+pack with the CPU oracle: masks, metadata and packed values
must be bit-identical for the same seed."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_10991_b200 import binding, workloads
from tests.helpers import layouts

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)
    return torch.from_numpy(a).to(DEV)


def gpu_prune(g_np, n, m, axis, seed, **kw):
    values, meta = binding.mvue_prune(to_dev(g_np), n, m, axis, seed, **kw)
    torch.cuda.synchronize()
    return values.view(torch.int16).cpu().numpy().view(np.uint16), meta.cpu().numpy()


def assert_parity(g_np, n, m, axis, seed, **kw):
    v_gpu, m_gpu = gpu_prune(g_np, n, m, axis, seed, **kw)
    v_ref, m_ref = oracle.prune(g_np, n, m, axis=axis, seed=seed, threads=oracle.host_threads(), **kw)
    assert v_gpu.shape == v_ref.shape and m_gpu.shape == m_ref.shape
    bad_m = np.flatnonzero(m_gpu.ravel() != m_ref.ravel())
    assert bad_m.size == 0, f"{bad_m.size} metadata bytes differ, first at {bad_m[:4]}"
    bad_v = np.flatnonzero(v_gpu.ravel() != v_ref.ravel())
    assert bad_v.size == 0, f"{bad_v.size} packed values differ, first at {bad_v[:4]}"


MODES = [(1, 2), (2, 4), (1, 4)]
# shapes span several thread blocks and leave ragged tails in both grid dimensions; the last three are made of whole
# 128 x 64 tiles, which the bf16 prune down the rows handles with a kernel of its own; (4096, 1024) and (176, 1536) are
# whole blocks of 16 rows x 512 columns, which the bf16 prune along the rows handles with a kernel of its own
SHAPES = [(16, 16), (48, 80), (528, 264), (1040, 1000), (4096, 1024), (256, 192), (1152, 320), (176, 1536),
          (512, 256), (256, 32), (384, 64), (192, 128),      # narrow K along the rows: several row groups per block
          (256, 768), (128, 640), (256, 576), (384, 1536)]   # down the rows: 12, 10, 9, 24 column tiles (tile walk orders)


@pytest.mark.parametrize("n,m", MODES)
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dist,dtype", [("relu_normal", "f32"), ("relu_lognormal", "bf16"),
                                        ("student_t", "bf16"), ("student_t", "f32")])
def test_bit_parity(n, m, axis, shape, dist, dtype):
    rows, cols = shape
    if axis == 1:                      # K = cols must be a multiple of 16, Mrows = rows of 8
        cols = (cols + 15) // 16 * 16
    else:
        rows, cols = (rows + 15) // 16 * 16, (cols + 7) // 8 * 8
    g = workloads.gradient((rows, cols), dist, seed=rows + cols, dtype=dtype)
    assert_parity(g, n, m, axis, seed=0x9E3779B97F4A7C15 ^ rows)


@pytest.mark.parametrize("n,m", MODES)
def test_linear_small_config(n, m):
    cfg = workloads.CONFIGS["linear_small"]
    g = workloads.gradient((cfg["T"], cfg["out"]), cfg["g_dist"], cfg["seed"], dtype="f32")
    assert_parity(g, n, m, axis=0, seed=0)
    assert_parity(g, n, m, axis=1, seed=0)


@pytest.mark.parametrize("n,m,joint", [(1, 2, None), (2, 4, binding.MVUE_JOINT_TABLE),
                                       (2, 4, binding.MVUE_JOINT_SYSTEMATIC), (2, 4, binding.MVUE_JOINT_APPROX),
                                       (1, 4, None)])
def test_linear_small_slice_is_unbiased_over_10k_seeds(n, m, joint):
    # the 16 x 16 slice of the small linear-layer gradient, pruned by the CUDA kernel under 10000 seeds: the mean of
    # the unpacked estimates must sit within six standard errors of the gradient, the standard error taken from the
    # estimator's own survival probabilities (Sec. 4.1 / 4.2 / 4.4)
    from oracle import theory
    cfg = workloads.CONFIGS["linear_small"]
    g = np.ascontiguousarray(
        workloads.gradient((cfg["T"], cfg["out"]), cfg["g_dist"], cfg["seed"], dtype="f32")[:16, :16])
    g_dev = to_dev(g)
    n_seeds = 10000
    acc = torch.zeros((16, 16), dtype=torch.float64, device=DEV)
    values = torch.empty((16, 8), dtype=torch.bfloat16, device=DEV)
    meta = torch.empty((16, 2), dtype=torch.uint8, device=DEV)
    for seed in range(n_seeds):
        binding.mvue_prune(g_dev, n, m, 0, seed, values=values, meta=meta, joint=joint)
        acc += binding.mvue_unpack(values, meta).double()
    mean = (acc / n_seeds).cpu().numpy()                                   # A = g^T: [16, 16]
    A = g.T.astype(np.float64)
    for r in range(16):
        for j in range(4):
            blk = A[r, 4 * j:4 * j + 4]
            if m == 2:
                p = np.zeros(4)
                for h in range(2):
                    s = abs(blk[2 * h]) + abs(blk[2 * h + 1])
                    if s > 0:
                        p[2 * h], p[2 * h + 1] = abs(blk[2 * h]) / s, abs(blk[2 * h + 1]) / s
            elif n == 1:                                                    # MVUE 1:4: p_i = |a_i| / S
                p = np.abs(blk) / max(np.abs(blk).sum(), 1e-300)
            elif np.count_nonzero(blk) < 2:
                p = (blk != 0).astype(np.float64)
            elif joint == binding.MVUE_JOINT_APPROX:
                p = theory.approx24_inclusion(blk)
            else:
                p = theory.marginals24(blk)
            for e in range(4):
                a = blk[e]
                if a == 0:
                    assert mean[r, 4 * j + e] == 0
                    continue
                sd = np.sqrt(a * a * max(1 / p[e] - 1, 0.0) / n_seeds)
                assert abs(mean[r, 4 * j + e] - a) <= 6 * sd + 2.0 ** -8 * abs(a), (r, j, e, mean[r, 4 * j + e], a)


@pytest.mark.parametrize("n,m", MODES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_edge_values(n, m, dtype):
    # all-zero groups, single non-zeros, ties, negative zeros, denormals, huge/tiny mixtures,
    # and blocks on the case boundaries a_4 = 2 a_1 + a_3 and a_4 = a_1 + a_2 + a_3
    rng = np.random.Generator(np.random.PCG64(17))
    pool = np.array([0.0, -0.0, 1.0, -1.0, 2.0, 3.0, 5.0, 6.0, 0.5, 1e-3, 1e3, 2.0**-126, 2.0**-133,
                     -2.0**-130, 2.0**100, -2.0**120, 1.5, 1.75, 3.0e-39], dtype=np.float32)
    g = pool[rng.integers(0, len(pool), size=(256, 128))]
    g[0, :8] = [1, 2, 3, 5, 1, 2, 3, 6]
    g[1, :8] = [0, 0, 0, 0, -0.0, -0.0, -0.0, -0.0]
    g[2, :8] = [2, 2, 2, 2, 0, 0, 0, 7]
    g[3, :8] = [3, -3, 3, -3, 0, 1, 1, 1]
    if dtype == "bf16":
        g = workloads.to_bf16_bits(g)
    for axis in (0, 1):
        for seed in (0, 1, 2**63 + 5):
            assert_parity(np.ascontiguousarray(g), n, m, axis, seed)


@pytest.mark.parametrize("n,m", MODES)
@pytest.mark.parametrize("axis", [0, 1])
def test_strided_input_and_k_shards(n, m, axis):
    full = workloads.gradient((256, 192), "student_t", seed=5, dtype="bf16")
    # a view with ld > cols
    sub = full[:, :128]
    g_dev = to_dev(full)[:, :128]
    assert g_dev.stride(0) == 192
    values, meta = binding.mvue_prune(g_dev, n, m, axis, 77)
    v_ref, m_ref = oracle.prune(np.ascontiguousarray(sub), n, m, axis=axis, seed=77)
    assert np.array_equal(values.view(torch.int16).cpu().numpy().view(np.uint16), v_ref)
    assert np.array_equal(meta.cpu().numpy(), m_ref)
    # shards of the K axis reproduce the unsharded masks
    g = np.ascontiguousarray(sub)
    K = g.shape[1] if axis == 1 else g.shape[0]
    v_all, m_all = gpu_prune(g, n, m, axis, 123)
    for lo, hi in [(0, 48), (48, K)]:
        part = g[:, lo:hi] if axis == 1 else g[lo:hi]
        v, mt = gpu_prune(np.ascontiguousarray(part), n, m, axis, 123, k_total=K, k_offset=lo)
        assert np.array_equal(v, v_all[:, lo // 2:hi // 2]) and np.array_equal(mt, m_all[:, lo // 8:hi // 8])
        assert_parity(np.ascontiguousarray(part), n, m, axis, 123, k_total=K, k_offset=lo)


@pytest.mark.parametrize("n,m", MODES)
def test_unpack_matches_oracle_unpack(n, m):
    g = workloads.gradient((128, 96), "relu_normal", seed=3, dtype="bf16")
    values, meta = binding.mvue_prune(to_dev(g), n, m, 1, 9)
    dense = binding.mvue_unpack(values, meta).float().cpu().numpy()
    v_ref, m_ref = oracle.prune(g, n, m, axis=1, seed=9)
    assert np.array_equal(dense, oracle.unpack(v_ref, m_ref))


def test_same_seed_same_bits_and_seed_matters():
    g = workloads.gradient((512, 512), "student_t", seed=8, dtype="bf16")
    a = gpu_prune(g, 2, 4, 0, 1)
    b = gpu_prune(g, 2, 4, 0, 1)
    c = gpu_prune(g, 2, 4, 0, 2)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert not np.array_equal(a[1], c[1])


def test_bad_arguments_launch_nothing():
    g = to_dev(workloads.gradient((64, 64), "student_t", seed=1, dtype="bf16"))
    for n, m, axis, status in [(3, 4, 1, -2), (2, 4, 3, -3)]:
        with pytest.raises(binding.MvueError) as e:
            binding.mvue_prune(g, n, m, axis, 0)
        assert e.value.status == status
    with pytest.raises(binding.MvueError) as e:
        binding.mvue_prune(g[:, :40], 2, 4, 1, 0)              # K = 40 is not a multiple of 16
    assert e.value.status == -3
    with pytest.raises(binding.MvueError) as e:
        binding.mvue_prune(g[:, 4:36], 2, 4, 1, 0)             # base pointer off the 16-byte grid
    assert e.value.status == -4


@pytest.mark.parametrize("name,n,m", [("conv_im2col", 2, 4), ("conv_im2col", 1, 2), ("ffn_768", 2, 4)])
def test_full_size_configs_sampled(name, n, m):
    """Full-size tensors in the launch shape the benchmark times; the oracle evaluates every
    block of a seeded sample of row strips (any block is computable alone: the generator is
    counter-based) and the whole tensor when it is small enough."""
    cfg = workloads.CONFIGS[name]
    g = workloads.gradient((cfg["T"], cfg["out"]), cfg["g_dist"], cfg["seed"], dtype="bf16")
    seed = 1000 + cfg["seed"]
    v_gpu, m_gpu = gpu_prune(g, n, m, 0, seed)
    T = cfg["T"]
    rng = np.random.Generator(np.random.PCG64(99))
    starts = sorted(set([0, T - 64] + [int(x) * 16 for x in rng.integers(0, T // 16 - 4, 40)]))
    for lo in starts:
        part = np.ascontiguousarray(g[lo:lo + 64])
        v_ref, m_ref = oracle.prune(part, n, m, axis=0, seed=seed, k_total=T, k_offset=lo)
        assert np.array_equal(v_gpu[:, lo // 2:lo // 2 + 32], v_ref)
        assert np.array_equal(m_gpu[:, lo // 8:lo // 8 + 8], m_ref)
    # properties that hold at any size
    lo2, hi2 = m_gpu & 3, (m_gpu >> 2) & 3
    assert (lo2 < hi2).all() and ((m_gpu >> 4) & 3 < (m_gpu >> 6) & 3).all()


@pytest.mark.parametrize("n,m", MODES)
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", [(128, 128), (384, 200), (1024, 136), (2048, 1000), (4096, 1024), (256, 768), (128, 640),
                                   (256, 1152)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_tensor_core_metadata_order(n, m, axis, shape, dtype):
    """layout = MVUE_LAYOUT_TC: same survivors, metadata bit-identical to the oracle's once carried into
    the tensor-core order (padding rows hold a valid pattern), and mvue_unpack reads it back."""
    rows, cols = shape
    if axis == 1:
        cols = (cols + 127) // 128 * 128
    else:
        rows, cols = (rows + 127) // 128 * 128, (cols + 7) // 8 * 8
    g = workloads.gradient((rows, cols), "relu_lognormal", seed=rows ^ cols, dtype=dtype)
    values, meta = binding.mvue_prune(to_dev(g), n, m, axis, 31, layout=binding.MVUE_LAYOUT_TC)
    dense = binding.mvue_unpack(values, meta, layout=binding.MVUE_LAYOUT_TC)
    torch.cuda.synchronize()
    v_ref, m_ref = oracle.prune(g, n, m, axis=axis, seed=31, threads=oracle.host_threads())
    assert np.array_equal(values.view(torch.int16).cpu().numpy().view(np.uint16), v_ref)
    got = meta.cpu().numpy().reshape(-1)
    want = layouts.canonical_to_tc(m_ref)
    assert got.shape == want.shape
    assert np.array_equal(got, want)
    assert np.array_equal(layouts.tc_to_canonical(got, *m_ref.shape[:1], m_ref.shape[1] * 8), m_ref)
    assert np.array_equal(dense.float().cpu().numpy(), oracle.unpack(v_ref, m_ref))


@pytest.mark.parametrize("axis", [0, 1])
def test_k_shards_in_tensor_core_order(axis):
    """A token shard pruned with the global block numbering: same survivors and masks as the slice of the
    unsharded run, metadata laid out for the shard's own K."""
    g = workloads.gradient((512, 384), "student_t", seed=6, dtype="bf16")
    K = g.shape[1] if axis == 1 else g.shape[0]
    v_all, m_all = oracle.prune(g, 2, 4, axis=axis, seed=55, threads=oracle.host_threads())
    for lo, hi in [(0, 128), (128, K)]:
        part = np.ascontiguousarray(g[:, lo:hi] if axis == 1 else g[lo:hi])
        values, meta = binding.mvue_prune(to_dev(part), 2, 4, axis, 55, k_total=K, k_offset=lo,
                                          layout=binding.MVUE_LAYOUT_TC)
        torch.cuda.synchronize()
        assert np.array_equal(values.view(torch.int16).cpu().numpy().view(np.uint16), v_all[:, lo // 2:hi // 2])
        want = layouts.canonical_to_tc(np.ascontiguousarray(m_all[:, lo // 8:hi // 8]))
        assert np.array_equal(meta.cpu().numpy().reshape(-1), want)

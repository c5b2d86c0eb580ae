"""Parity of the CUDA prune+pack with the CPU oracle for the 2:4 estimators chosen through
mvue_prune_joint (systematic sampling; approx-MVUE of Sec. 4.4): masks, metadata and packed values
bit-identical for the same seed."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_10991_b200 import binding, workloads
from tests.helpers import layouts

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
SYS = binding.MVUE_JOINT_SYSTEMATIC
APPROX = binding.MVUE_JOINT_APPROX
JOINTS = [SYS, APPROX]              # the binding's and the oracle's codes agree (0, 1, 2)


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)
    return torch.from_numpy(a).to(DEV)


def gpu_prune(g_np, axis, seed, joint=SYS, n=2, m=4, **kw):
    values, meta = binding.mvue_prune(to_dev(g_np), n, m, axis, seed, joint=joint, **kw)
    torch.cuda.synchronize()
    return values.view(torch.int16).cpu().numpy().view(np.uint16), meta.cpu().numpy()


def assert_parity(g_np, axis, seed, joint=SYS, **kw):
    v_gpu, m_gpu = gpu_prune(g_np, axis, seed, joint=joint, **kw)
    v_ref, m_ref = oracle.prune(g_np, 2, 4, axis=axis, seed=seed, threads=oracle.host_threads(),
                                joint={SYS: oracle.JOINT_SYSTEMATIC, APPROX: oracle.JOINT_APPROX}[joint], **kw)
    assert v_gpu.shape == v_ref.shape and m_gpu.shape == m_ref.shape
    bad_m = np.flatnonzero(m_gpu.ravel() != m_ref.ravel())
    assert bad_m.size == 0, f"{bad_m.size} metadata bytes differ, first at {bad_m[:4]}"
    bad_v = np.flatnonzero(v_gpu.ravel() != v_ref.ravel())
    assert bad_v.size == 0, f"{bad_v.size} packed values differ, first at {bad_v[:4]}"


# shapes span several thread blocks and leave ragged tails in both grid dimensions; the last three are made of whole
# 128 x 64 tiles, which the bf16 prune down the rows handles with a kernel of its own; (4096, 1024) and (176, 1536) are
# whole blocks of 16 rows x 512 columns, which the bf16 prune along the rows handles with a kernel of its own
SHAPES = [(16, 16), (48, 80), (528, 264), (1040, 1000), (4096, 1024), (256, 192), (1152, 320), (176, 1536)]


@pytest.mark.parametrize("joint", JOINTS)
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dist,dtype", [("relu_normal", "f32"), ("relu_lognormal", "bf16"),
                                        ("student_t", "bf16"), ("student_t", "f32")])
def test_bit_parity(axis, shape, dist, dtype, joint):
    rows, cols = shape
    if axis == 1:
        cols = (cols + 15) // 16 * 16
    else:
        rows, cols = (rows + 15) // 16 * 16, (cols + 7) // 8 * 8
    g = workloads.gradient((rows, cols), dist, seed=rows + cols, dtype=dtype)
    assert_parity(g, axis, seed=0x9E3779B97F4A7C15 ^ rows, joint=joint)


@pytest.mark.parametrize("joint", JOINTS)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_edge_values(dtype, joint):
    # all-zero groups, lone non-zeros in every position, exactly-half and empty intervals, ties, negative
    # zeros, denormals (the lone-non-zero rule rests on 2^-149 surviving an addition), huge/tiny mixtures
    rng = np.random.Generator(np.random.PCG64(19))
    pool = np.array([0.0, -0.0, 1.0, -1.0, 2.0, 3.0, 5.0, 6.0, 0.5, 1e-3, 1e3, 2.0**-126, 2.0**-133,
                     -2.0**-130, 2.0**100, -2.0**120, 1.5, 1.75, 3.0e-39], dtype=np.float32)
    g = pool[rng.integers(0, len(pool), size=(256, 128))]
    g[0, :16] = [1, 2, 3, 4, 1, -1, -10, 1, 10, 1, 1, 1, 1, 10, 1, 1]
    g[1, :16] = [0, 0, 0, 0, -0.0, -0.0, -0.0, -0.0, 5, 0, 0, 0, 0, -5, 0, 0]
    g[2, :16] = [0, 0, 5, 0, 0, 0, 0, -5, 1, 0, 0, 1, 1, 1, 0, 0]
    g[3, :16] = [3, -3, 3, -3, 0, 1, 1, 1, 0, 2, 2, 0, 3, 0, 3, 0]
    g[4, :8] = [2.0**-140, 0, 0, 0, 0, 0, 2.0**-149, 2.0**-149]
    if dtype == "bf16":
        g = workloads.to_bf16_bits(g)
    for axis in (0, 1):
        for seed in (0, 1, 2**63 + 5):
            assert_parity(np.ascontiguousarray(g), axis, seed, joint=joint)


@pytest.mark.parametrize("joint", JOINTS)
@pytest.mark.parametrize("axis", [0, 1])
def test_strided_input_and_k_shards(axis, joint):
    full = workloads.gradient((256, 192), "student_t", seed=5, dtype="bf16")
    sub = full[:, :128]
    g_dev = to_dev(full)[:, :128]
    values, meta = binding.mvue_prune(g_dev, 2, 4, axis, 77, joint=joint)
    v_ref, m_ref = oracle.prune(np.ascontiguousarray(sub), 2, 4, axis=axis, seed=77, joint=joint)
    assert np.array_equal(values.view(torch.int16).cpu().numpy().view(np.uint16), v_ref)
    assert np.array_equal(meta.cpu().numpy(), m_ref)
    g = np.ascontiguousarray(sub)
    K = g.shape[1] if axis == 1 else g.shape[0]
    v_all, m_all = gpu_prune(g, axis, 123, joint=joint)
    for lo, hi in [(0, 48), (48, K)]:
        part = np.ascontiguousarray(g[:, lo:hi] if axis == 1 else g[lo:hi])
        v, mt = gpu_prune(part, axis, 123, joint=joint, k_total=K, k_offset=lo)
        assert np.array_equal(v, v_all[:, lo // 2:hi // 2]) and np.array_equal(mt, m_all[:, lo // 8:hi // 8])
        assert_parity(part, axis, 123, joint=joint, k_total=K, k_offset=lo)


@pytest.mark.parametrize("joint", JOINTS)
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape", [(128, 128), (384, 200), (2048, 1000)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_tensor_core_metadata_order(axis, shape, dtype, joint):
    rows, cols = shape
    if axis == 1:
        cols = (cols + 127) // 128 * 128
    else:
        rows, cols = (rows + 127) // 128 * 128, (cols + 7) // 8 * 8
    g = workloads.gradient((rows, cols), "relu_lognormal", seed=rows ^ cols, dtype=dtype)
    values, meta = binding.mvue_prune(to_dev(g), 2, 4, axis, 31, layout=binding.MVUE_LAYOUT_TC, joint=joint)
    dense = binding.mvue_unpack(values, meta, layout=binding.MVUE_LAYOUT_TC)
    torch.cuda.synchronize()
    v_ref, m_ref = oracle.prune(g, 2, 4, axis=axis, seed=31, threads=oracle.host_threads(), joint=joint)
    assert np.array_equal(values.view(torch.int16).cpu().numpy().view(np.uint16), v_ref)
    assert np.array_equal(meta.cpu().numpy().reshape(-1), layouts.canonical_to_tc(m_ref))
    assert np.array_equal(dense.float().cpu().numpy(), oracle.unpack(v_ref, m_ref))


def test_the_laws_differ_and_one_of_two_ignores_the_choice():
    g = workloads.gradient((512, 512), "student_t", seed=8, dtype="bf16")
    tab = gpu_prune(g, 0, 1, joint=binding.MVUE_JOINT_TABLE)
    dflt = binding.mvue_prune(to_dev(g), 2, 4, 0, 1)
    assert np.array_equal(tab[1], dflt[1].cpu().numpy())           # mvue_prune is the table law
    sys_ = gpu_prune(g, 0, 1)
    apx = gpu_prune(g, 0, 1, joint=APPROX)
    assert not np.array_equal(tab[1], sys_[1]) and not np.array_equal(tab[1], apx[1])
    assert not np.array_equal(sys_[1], apx[1])
    a = gpu_prune(g, 1, 3, joint=binding.MVUE_JOINT_TABLE, n=1, m=2)
    for joint in JOINTS:
        b = gpu_prune(g, 1, 3, joint=joint, n=1, m=2)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_unknown_joint_is_rejected():
    g = to_dev(workloads.gradient((64, 64), "student_t", seed=1, dtype="bf16"))
    for joint in (3, -1):
        with pytest.raises(binding.MvueError) as e:
            binding.mvue_prune(g, 2, 4, 1, 0, joint=joint)
        assert e.value.status == -11


@pytest.mark.parametrize("joint", JOINTS)
def test_full_size_conv_im2col_sampled(joint):
    cfg = workloads.CONFIGS["conv_im2col"]
    g = workloads.gradient((cfg["T"], cfg["out"]), cfg["g_dist"], cfg["seed"], dtype=cfg["g_dtype"])
    seed = 4321
    values, meta = binding.mvue_prune(to_dev(g), 2, 4, 0, seed, layout=binding.MVUE_LAYOUT_TC, joint=joint)
    torch.cuda.synchronize()
    v_gpu = values.view(torch.int16).cpu().numpy().view(np.uint16)
    T = cfg["T"]
    m_gpu = layouts.tc_to_canonical(meta.cpu().numpy().reshape(-1), cfg["out"], T)
    rng = np.random.Generator(np.random.PCG64(5))
    starts = sorted(set([0, T - 128] + [int(x) * 128 for x in rng.integers(0, T // 128 - 1, 40)]))
    for lo in starts:
        part = np.ascontiguousarray(g[lo:lo + 128])
        v_ref, m_ref = oracle.prune(part, 2, 4, axis=0, seed=seed, k_total=T, k_offset=lo, joint=joint)
        assert np.array_equal(v_gpu[:, lo // 2:lo // 2 + 64], v_ref)
        assert np.array_equal(m_gpu[:, lo // 8:lo // 8 + 16], m_ref)

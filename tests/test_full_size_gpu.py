"""The benchmark's workloads at full size, in the launch configuration `bench.py` times: prune+pack in
tensor-core order followed by the sparse update product.  The oracle prunes the whole gradient (every
block is independent), and the product is checked on whole rows of A that it can afford plus a seeded
sample of single entries computed one by one in fp64."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_10991_b200 import binding, workloads
from tests.helpers import layouts

pytestmark = pytest.mark.gpu
TC = binding.MVUE_LAYOUT_TC


def to_dev(a):
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("name,n,m,check_rows", [("conv_im2col", 2, 4, 2), ("conv_im2col", 1, 2, 1),
                                                 ("ffn_large", 2, 4, 1)])
def test_bench_workload_full_size(name, n, m, check_rows):
    cfg = workloads.CONFIGS[name]
    T, n_out, n_in = cfg["T"], cfg["out"], cfg["inp"]
    g = workloads.gradient((T, n_out), cfg["g_dist"], cfg["seed"], dtype="bf16")
    h = workloads.normal_bf16((T, n_in), cfg["seed"] + 100)
    seed = 4242
    g_dev, h_dev = to_dev(g), to_dev(h)
    values, meta = binding.mvue_prune(g_dev, n, m, 0, seed, layout=TC)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dW = binding.mvue_sparse_update_gemm(values, meta, h_dev, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    th = oracle.host_threads()
    v_ref, m_ref = oracle.prune(g, n, m, axis=0, seed=seed, threads=th)
    # prune+pack: every survivor and every metadata byte of the full tensor
    assert np.array_equal(values.view(torch.int16).cpu().numpy().view(np.uint16), v_ref)
    assert np.array_equal(meta.cpu().numpy().reshape(-1), layouts.canonical_to_tc(m_ref))

    got = dW.double().cpu().numpy()
    rng = np.random.Generator(np.random.PCG64(7))
    rows = sorted(set([0, n_out - 1] + [int(x) for x in rng.integers(0, n_out, check_rows)]))
    A_rows = oracle.unpack(np.ascontiguousarray(v_ref[rows]), np.ascontiguousarray(m_ref[rows]))
    # whole rows on a column panel the plain loops can afford
    panel = np.ascontiguousarray(h[:, :64])
    want = oracle.gemm(A_rows, panel, threads=th)
    err = np.linalg.norm(got[rows][:, :64] - want) / np.linalg.norm(want)
    assert err <= 1e-2 and err <= 5e-5, err
    # single entries anywhere in the output
    for i_r, r in enumerate(rows):
        for j in [int(x) for x in rng.integers(0, n_in, 12)]:
            w = oracle.gemm_entry(A_rows[i_r], h, j)
            scale = float(np.abs(A_rows[i_r]).sum()) * 3.0
            assert abs(got[r, j] - w) <= 1e-5 * scale + 1e-4 * abs(w), (r, j, got[r, j], w)
    if n_out * n_in >= 1 << 24:
        # an output of hundreds of tiles (persistent walk in bands, last round cut along K): the whole first 256-row
        # tile and the whole last one -- the last tiles in tile order are the ones a partly filled round splits --
        # on the first and the last 64 columns, and 500 entries scattered over the whole output
        for r0 in (0, n_out - 256):
            block = list(range(r0, r0 + 256))
            A_blk = oracle.unpack(np.ascontiguousarray(v_ref[block]), np.ascontiguousarray(m_ref[block]))
            for c0 in (0, n_in - 64):
                want = oracle.gemm(A_blk, np.ascontiguousarray(h[:, c0:c0 + 64]), threads=th)
                err = np.linalg.norm(got[r0:r0 + 256, c0:c0 + 64] - want) / np.linalg.norm(want)
                assert err <= 5e-5, (r0, c0, err)
                assert np.abs(got[r0:r0 + 256, c0:c0 + 64] - want).max() <= 1e-3 * np.abs(want).max(), (r0, c0)
        cache = {}
        for r, j in zip(rng.integers(0, n_out, 500), rng.integers(0, n_in, 500)):
            r, j = int(r), int(j)
            if r not in cache:
                cache[r] = oracle.unpack(np.ascontiguousarray(v_ref[r:r + 1]), np.ascontiguousarray(m_ref[r:r + 1]))[0]
            w = oracle.gemm_entry(cache[r], h, j)
            scale = float(np.abs(cache[r]).sum()) * 3.0
            assert abs(got[r, j] - w) <= 1e-5 * scale + 1e-4 * abs(w), (r, j, got[r, j], w)


def test_mlp_stack_block_full_size():
    """One block of the MLP-stack workload at full size (T = 32768, d = 1024, d_ff = 4096): the two layers' four
    prunes bit for bit over the whole tensors, and the two update and two backward products (f'(z) epilogue, bf16
    out) on seeded samples computed entry by entry in fp64.  Each layer is checked on the gradient the GPU chain
    actually propagated, so a mismatch names the step that made it."""
    cfg = workloads.CONFIGS["mlp_stack"]
    T, d_ff, d = cfg["T"], cfg["out"], cfg["inp"]
    th = oracle.host_threads()
    rng = np.random.Generator(np.random.PCG64(11))
    g_np = workloads.gradient((T, d), cfg["g_dist"], cfg["seed"], dtype="bf16")
    for layer, (n_out, n_in) in enumerate([(d, d_ff), (d_ff, d)]):
        W = workloads.normal_bf16((n_out, n_in), seed=50 + layer, std=n_in ** -0.5)
        h = workloads.normal_bf16((T, n_in), seed=60 + layer)
        act = workloads.normal_bf16((T, n_in), seed=70 + layer)
        g_dev, W_dev, h_dev, act_dev = to_dev(g_np), to_dev(W), to_dev(h), to_dev(act)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        s_upd, s_bwd = 1000 + 2 * layer, 1001 + 2 * layer
        v0, m0 = binding.mvue_prune(g_dev, 2, 4, 0, s_upd, layout=TC)
        dW = binding.mvue_sparse_update_gemm(v0, m0, h_dev, dev_status=status)
        v1, m1 = binding.mvue_prune(g_dev, 2, 4, 1, s_bwd, layout=TC)
        dh = binding.mvue_sparse_backward_gemm(v1, m1, W_dev, act_grad=act_dev, out_dtype=torch.bfloat16,
                                               dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0

        # the four packed operands, whole
        v0_ref, m0_ref = oracle.prune(g_np, 2, 4, axis=0, seed=s_upd, threads=th)
        v1_ref, m1_ref = oracle.prune(g_np, 2, 4, axis=1, seed=s_bwd, threads=th)
        assert np.array_equal(v0.view(torch.int16).cpu().numpy().view(np.uint16), v0_ref)
        assert np.array_equal(m0.cpu().numpy().reshape(-1), layouts.canonical_to_tc(m0_ref))
        assert np.array_equal(v1.view(torch.int16).cpu().numpy().view(np.uint16), v1_ref)
        assert np.array_equal(m1.cpu().numpy().reshape(-1), layouts.canonical_to_tc(m1_ref))

        # update product dW[n_out x n_in]: sampled entries
        got = dW.double().cpu().numpy()
        rows = sorted(set([0, n_out - 1] + [int(x) for x in rng.integers(0, n_out, 2)]))
        A_rows = oracle.unpack(np.ascontiguousarray(v0_ref[rows]), np.ascontiguousarray(m0_ref[rows]))
        for i_r, r in enumerate(rows):
            for j in [0, n_in - 1] + [int(x) for x in rng.integers(0, n_in, 6)]:
                w = oracle.gemm_entry(A_rows[i_r], h, j)
                scale = float(np.abs(A_rows[i_r]).sum()) * 3.0
                assert abs(got[r, j] - w) <= 1e-5 * scale + 1e-4 * abs(w), ("dW", layer, r, j, got[r, j], w)

        # backward product dh[T x n_in] = (theta(g) W) * f'(z), stored as bf16: sampled entries (first and last tile
        # rows and columns among them) within bf16 rounding of the fp64 value
        dh_np = dh.view(torch.int16).cpu().numpy().view(np.uint16)
        got_h = oracle.bf16_to_f32(dh_np).astype(np.float64)
        t_rows = sorted(set([0, 127, 128, 255, 256, T - 1] + [int(x) for x in rng.integers(0, T, 10)]))
        A_t = oracle.unpack(np.ascontiguousarray(v1_ref[t_rows]), np.ascontiguousarray(m1_ref[t_rows]))
        act_f = oracle.bf16_to_f32(act).astype(np.float64)
        for i_r, r in enumerate(t_rows):
            for j in [0, 15, 16, 63, 64, 127, 128, 255, 256, n_in - 1] + [int(x) for x in rng.integers(0, n_in, 6)]:
                w = oracle.gemm_entry(A_t[i_r], W, j) * act_f[r, j]
                scale = float(np.abs(A_t[i_r]).sum()) * float(n_in ** -0.5) * 3.0 * abs(act_f[r, j])
                assert abs(got_h[r, j] - w) <= 2.0 ** -8 * abs(w) + 1e-5 * scale, ("dh", layer, r, j, got_h[r, j], w)
        g_np = np.ascontiguousarray(dh_np)                  # the next layer sees what the GPU stored
        del g_dev, W_dev, h_dev, act_dev, v0, m0, v1, m1, dW, dh
        torch.cuda.empty_cache()


@pytest.mark.parametrize("axis", [0, 1])
def test_prune_4gb_tensor_sampled(axis):
    """The largest tensor of the bandwidth sweep, bf16 [524288 x 4096] = 4 GiB (element offsets reach 2^31, byte
    offsets 2^32): seeded slices of the packed output against the oracle, which prunes any block on its own because
    the random words are a function of the block number.  The tensor is 16 copies of a 256 MiB seeded base stacked
    along the rows (as in the sweep), so a slice's input is known on the host without moving 4 GiB."""
    rows, cols, base_rows = 1 << 19, 4096, 1 << 15
    base = workloads.gradient((base_rows, cols), "student_t", 5, dtype="bf16")
    g_dev = to_dev(base).repeat(rows // base_rows, 1)
    assert g_dev.shape == (rows, cols) and g_dev.is_contiguous()
    seed = 99
    rng = np.random.Generator(np.random.PCG64(3))
    for n, m in ((2, 4), (1, 2)):
        values, meta = binding.mvue_prune(g_dev, n, m, axis, seed)            # canonical layout
        torch.cuda.synchronize()
        starts = sorted(set([0, rows - 128, rows // 2, rows // 2 + 128] +
                            [int(x) * 128 for x in rng.integers(0, rows // 128, 6)]))
        for lo in starts:
            part = np.ascontiguousarray(base[np.arange(lo, lo + 128) % base_rows])
            if axis == 1:      # A = g: rows lo .. lo+127 of A; block numbers depend on the global row
                # the oracle's tensor call numbers blocks from row 0 of what it is given, so rows far down the
                # tensor are checked through per-block calls with their global block numbers
                v_gpu = values[lo:lo + 128].view(torch.int16).cpu().numpy().view(np.uint16)
                m_gpu = meta[lo:lo + 128].cpu().numpy()
                for r in (0, 1, 63, 127):
                    for j in (0, 1, 511, 1023):
                        blk = oracle.bf16_to_f32(part[r, 4 * j:4 * j + 4])
                        nib = (int(m_gpu[r, j // 2]) >> (4 * (j % 2))) & 0xF
                        got = oracle.bf16_to_f32(v_gpu[r, 2 * j:2 * j + 2])
                        if m == 4:
                            idx, val = oracle.mvue_2of4(blk, oracle.block_word(seed, (lo + r) * (cols // 4) + j))
                        else:
                            idx, val = [], []
                            for half in range(2):
                                i1, v1 = oracle.mvue_1of2(float(blk[2 * half]), float(blk[2 * half + 1]),
                                                          oracle.block_word(seed, (lo + r) * (cols // 2) + 2 * j + half))
                                idx.append(2 * half + i1)
                                val.append(v1)
                        assert nib == idx[0] | (idx[1] << 2), (lo, r, j)
                        want = oracle.bf16_to_f32(oracle.bf16_rne(np.array(val, dtype=np.float32)))
                        assert np.array_equal(got, want), (lo, r, j)
            else:              # A = g^T: a K shard [lo, lo + 128) of every row of A
                v_ref, m_ref = oracle.prune(part, n, m, axis=0, seed=seed, k_total=rows, k_offset=lo,
                                            threads=oracle.host_threads())
                v_gpu = values[:, lo // 2:lo // 2 + 64].contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
                m_gpu = meta[:, lo // 8:lo // 8 + 16].contiguous().cpu().numpy()
                assert np.array_equal(v_gpu, v_ref), lo
                assert np.array_equal(m_gpu, m_ref), lo
        del values, meta
    del g_dev
    torch.cuda.empty_cache()


@pytest.mark.parametrize("axis", [0, 1])
def test_prune_4gb_tensor_sampled_in_the_sweeps_configuration(axis):
    """The same 4 GiB tensor as the bandwidth sweep launches it: systematic sampling, sixteen random bits per block,
    metadata in tensor-core order (down the rows this is the whole-tile kernel walking groups of eight column tiles;
    along the rows the whole-block kernel).  Seeded slices against the oracle: K shards of 128 rows down the rows,
    single rows with their global block numbers along the rows."""
    rows, cols, base_rows = 1 << 19, 4096, 1 << 15
    base = workloads.gradient((base_rows, cols), "student_t", 5, dtype="bf16")
    g_dev = to_dev(base).repeat(rows // base_rows, 1)
    seed, joint = 1234, binding.MVUE_JOINT_SYSTEMATIC
    values, meta = binding.mvue_prune(g_dev, 2, 4, axis, seed, layout=TC, joint=joint, options=binding.MVUE_OPT_EPS16)
    torch.cuda.synchronize()
    meta_flat = meta.reshape(-1)
    rng = np.random.Generator(np.random.PCG64(8))
    starts = sorted(set([0, rows - 128, rows // 2 - 128, rows // 2] + [int(x) * 128 for x in rng.integers(0, rows // 128, 6)]))
    th = oracle.host_threads()
    for lo in starts:
        part = np.ascontiguousarray(base[np.arange(lo, lo + 128) % base_rows])
        if axis == 0:          # A = g^T [cols x rows]: the K block lo / 128 of every row block of A
            v_ref, m_ref = oracle.prune(part, 2, 4, axis=0, seed=seed, k_total=rows, k_offset=lo, joint=joint, eps16=True,
                                        threads=th)
            v_gpu = values.view(cols, rows // 2)[:, lo // 2:lo // 2 + 64].contiguous().view(torch.int16).cpu().numpy()
            assert np.array_equal(v_gpu.view(np.uint16), v_ref), lo
            kblocks, kb = rows // 128, lo // 128
            blocks = torch.stack([meta_flat[(rb * kblocks + kb) * 2048:(rb * kblocks + kb + 1) * 2048]
                                  for rb in range(cols // 128)]).cpu().numpy()
            assert np.array_equal(layouts.tc_to_canonical(blocks, cols, 128), m_ref), lo
        else:                  # A = g: the row block lo / 128 with all its K blocks is contiguous in tensor-core order
            kblocks, rb = cols // 128, lo // 128
            m_gpu = layouts.tc_to_canonical(meta_flat[rb * kblocks * 2048:(rb + 1) * kblocks * 2048].cpu().numpy(), 128, cols)
            v_gpu = values.view(rows, cols // 2)[lo:lo + 128].view(torch.int16).cpu().numpy().view(np.uint16)
            for r in (0, 7, 8, 64, 127):
                v1, m1 = oracle.prune(np.ascontiguousarray(part[r:r + 1]), 2, 4, axis=1, seed=seed, joint=joint, eps16=True,
                                      k_total=cols * (lo + r + 1), k_offset=cols * (lo + r))
                assert np.array_equal(v_gpu[r], v1[0]), (lo, r)
                assert np.array_equal(m_gpu[r], m1[0]), (lo, r)
    del values, meta, g_dev
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name", ["conv_im2col", "ffn_large"])
@pytest.mark.parametrize("axis", [0, 1])
def test_bench_step_prune_full_size(name, axis):
    """The prune exactly as `bench.py`'s step and riders launch it (systematic sampling, sixteen random bits per block,
    tensor-core order), both orientations, on the whole tensor: every survivor and every metadata byte."""
    cfg = workloads.CONFIGS[name]
    T, n_out = cfg["T"], cfg["out"]
    g = workloads.gradient((T, n_out), cfg["g_dist"], cfg["seed"], dtype="bf16")
    seed, joint = 77, binding.MVUE_JOINT_SYSTEMATIC
    values, meta = binding.mvue_prune(to_dev(g), 2, 4, axis, seed, layout=TC, joint=joint, options=binding.MVUE_OPT_EPS16)
    torch.cuda.synchronize()
    v_ref, m_ref = oracle.prune(g, 2, 4, axis=axis, seed=seed, joint=joint, eps16=True, threads=oracle.host_threads())
    assert np.array_equal(values.view(torch.int16).cpu().numpy().view(np.uint16).reshape(v_ref.shape), v_ref)
    assert np.array_equal(meta.cpu().numpy().reshape(-1), layouts.canonical_to_tc(m_ref))

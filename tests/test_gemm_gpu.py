"""Parity of the 2:4-sparse tensor-core products with the CPU oracle (fp64 plain-loop product of the
oracle's own packed operand): relative Frobenius error <= 1e-2 for bf16 inputs with fp32
accumulation (the kernel is in fact exact to ~1e-6: bf16 products are exact in fp32)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_10991_b200 import binding, workloads
from tests.helpers import layouts

TC = binding.MVUE_LAYOUT_TC

pytestmark = pytest.mark.gpu
TOL = 1e-2          # the stated bar
TIGHT = 2e-5        # what fp32 accumulation of exact products actually gives at these K


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def rel_fro(got, want):
    return np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300)


def pack_canonical(A: np.ndarray):
    """Test-side packer for a hand-made 2:4 matrix (at most two non-zeros per group of four)."""
    M, K = A.shape
    vals = np.zeros((M, K // 2), dtype=np.float32)
    meta = np.zeros((M, K // 8), dtype=np.uint8)
    for r in range(M):
        for j in range(K // 4):
            nz = [i for i in range(4) if A[r, 4 * j + i] != 0]
            assert len(nz) <= 2
            idx = sorted(nz + [i for i in range(4) if i not in nz][:2 - len(nz)])
            vals[r, 2 * j], vals[r, 2 * j + 1] = A[r, 4 * j + idx[0]], A[r, 4 * j + idx[1]]
            meta[r, j // 2] |= (idx[0] | (idx[1] << 2)) << (4 * (j % 2))
    return workloads.to_bf16_bits(vals), meta


def test_one_hot_probes_fix_every_layout():
    # a single non-zero in A and in B: any mistake in the operand layouts, the metadata placement or
    # the output mapping moves or loses the single product
    M, N, K = 256, 512, 384
    rng = np.random.Generator(np.random.PCG64(3))
    for _ in range(24):
        m, n, k = int(rng.integers(0, M)), int(rng.integers(0, N)), int(rng.integers(0, K))
        A = np.zeros((M, K), dtype=np.float32)
        B = np.zeros((K, N), dtype=np.float32)
        A[m, k] = 2.0
        B[k, n] = -3.0
        vals, meta = pack_canonical(A)
        assert np.array_equal(oracle.unpack(vals, meta), A)
        out = binding.mvue_sparse_update_gemm(to_dev(vals), torch.from_numpy(layouts.canonical_to_tc(meta)).cuda(),
                                              to_dev(workloads.to_bf16_bits(B)))
        got = out.cpu().numpy()
        want = np.zeros((M, N), dtype=np.float32)
        want[m, n] = -6.0
        assert np.array_equal(got, want), (m, n, k, np.argwhere(got != 0)[:4])


@pytest.mark.parametrize("T,n_out,n_in", [(128, 8, 8), (512, 256, 256), (640, 136, 264), (2048, 384, 520),
                                          (8192, 768, 3072), (16384, 256, 2304)])
@pytest.mark.parametrize("n,m", [(2, 4), (1, 2), (1, 4)])
def test_update_gemm_matches_oracle(T, n_out, n_in, n, m):
    g = workloads.gradient((T, n_out), "student_t", seed=T + n_out, dtype="bf16")
    h = workloads.normal_bf16((T, n_in), seed=7)
    vals, meta = binding.mvue_prune(to_dev(g), n, m, 0, seed=11, layout=TC)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    dW = binding.mvue_sparse_update_gemm(vals, meta, to_dev(h), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    v_ref, m_ref = oracle.prune(g, n, m, axis=0, seed=11, threads=oracle.host_threads())
    A = oracle.unpack(v_ref, m_ref)
    if T * n_out * n_in <= 2 ** 31:
        want = oracle.gemm(A, h, threads=oracle.host_threads())
        err = rel_fro(dW.double().cpu().numpy(), want)
        assert err <= TOL and err <= TIGHT, err
    else:
        # too large for the plain loops: whole rows and columns, plus a seeded sample of entries
        got = dW.double().cpu().numpy()
        rng = np.random.Generator(np.random.PCG64(5))
        rows = [0, n_out - 1] + [int(x) for x in rng.integers(0, n_out, 6)]
        want_rows = oracle.gemm(A[rows], h, threads=oracle.host_threads())
        assert rel_fro(got[rows], want_rows) <= TIGHT
        for _ in range(200):
            i, j = int(rng.integers(0, n_out)), int(rng.integers(0, n_in))
            w = oracle.gemm_entry(A[i], h, j)
            assert abs(got[i, j] - w) <= 1e-4 * (abs(w) + np.abs(A[i]).sum() * 1e-3)


@pytest.mark.parametrize("T,n_out,n_in", [(256, 512, 128), (1000, 768, 3072), (8192, 3072, 768)])
@pytest.mark.parametrize("with_act", [False, True])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_backward_gemm_matches_oracle(T, n_out, n_in, with_act, out_dtype):
    g = workloads.gradient((T, n_out), "student_t", seed=3, dtype="bf16")
    W = workloads.normal_bf16((n_out, n_in), seed=4, std=0.02)
    act = workloads.normal_bf16((T, n_in), seed=5) if with_act else None
    vals, meta = binding.mvue_prune(to_dev(g), 2, 4, 1, seed=21, layout=TC)
    dh = binding.mvue_sparse_backward_gemm(vals, meta, to_dev(W), act_grad=None if act is None else to_dev(act),
                                           out_dtype=out_dtype)
    v_ref, m_ref = oracle.prune(g, 2, 4, axis=1, seed=21, threads=oracle.host_threads())
    A = oracle.unpack(v_ref, m_ref)
    rows = np.arange(T) if T * n_out * n_in <= 2 ** 30 else np.random.Generator(np.random.PCG64(1)).integers(0, T, 64)
    want = oracle.gemm(A[rows], W, None if act is None else act[rows], threads=oracle.host_threads())
    err = rel_fro(dh.double().cpu().numpy()[rows], want)
    assert err <= TOL
    assert err <= (TIGHT if out_dtype == torch.float32 else 4e-3), err


@pytest.mark.parametrize("T,n_out,n_in", [(8192 + 72, 1024, 4104), (4096, 2048, 520), (20000, 128, 1280)])
@pytest.mark.parametrize("with_act", [False, True])
def test_short_k_bf16_products_with_many_tiles(T, n_out, n_in, with_act):
    # bf16 outputs over a short reduction axis: every pair of blocks walks through several tiles back to back (the
    # hand-over of the accumulator between tiles is most of what such a product waits for), the last row and column tiles
    # are ragged, and the same product written as fp32 must round to the same bf16 numbers
    g = workloads.gradient((T, n_out), "student_t", seed=31, dtype="bf16")
    W = workloads.normal_bf16((n_out, n_in), seed=32, std=n_out ** -0.5)
    act = workloads.normal_bf16((T, n_in), seed=33) if with_act else None
    act_dev = None if act is None else to_dev(act)
    vals, meta = binding.mvue_prune(to_dev(g), 2, 4, 1, seed=34, layout=TC, joint=binding.MVUE_JOINT_SYSTEMATIC)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dh = binding.mvue_sparse_backward_gemm(vals, meta, to_dev(W), act_grad=act_dev, out_dtype=torch.bfloat16,
                                           dev_status=status)
    ref32 = binding.mvue_sparse_backward_gemm(vals, meta, to_dev(W), act_grad=act_dev, out_dtype=torch.float32,
                                              dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(dh.view(torch.int16), ref32.to(torch.bfloat16).view(torch.int16))
    v_ref, m_ref = oracle.prune(g, 2, 4, axis=1, seed=34, threads=oracle.host_threads(), joint=oracle.JOINT_SYSTEMATIC)
    rows = np.array(sorted({0, 127, 128, 255, 256, T - 1, T - 9} | set(
        np.random.Generator(np.random.PCG64(2)).integers(0, T, 40).tolist())))
    A = oracle.unpack(np.ascontiguousarray(v_ref[rows]), np.ascontiguousarray(m_ref[rows]))
    want = oracle.gemm(A, W, None if act is None else np.ascontiguousarray(act[rows]), threads=oracle.host_threads())
    err = rel_fro(dh.double().cpu().numpy()[rows], want)
    assert err <= 4e-3, err


def test_accumulate_and_preallocated_output():
    T, n_out, n_in = 1024, 256, 512
    g = workloads.gradient((T, n_out), "relu_lognormal", seed=1, dtype="bf16")
    h = workloads.normal_bf16((T, n_in), seed=2)
    vals, meta = binding.mvue_prune(to_dev(g), 2, 4, 0, seed=1, layout=TC)
    once = binding.mvue_sparse_update_gemm(vals, meta, to_dev(h))
    acc = torch.full((n_out, n_in), 1.5, dtype=torch.float32, device="cuda")
    binding.mvue_sparse_update_gemm(vals, meta, to_dev(h), out=acc, accumulate=True)
    assert torch.allclose(acc, once + 1.5, rtol=1e-6, atol=1e-6)
    # a strided output view
    big = torch.zeros((n_out, n_in + 64), dtype=torch.float32, device="cuda")
    binding.mvue_sparse_update_gemm(vals, meta, to_dev(h), out=big[:, :n_in])
    assert torch.equal(big[:, :n_in], once) and float(big[:, n_in:].abs().sum()) == 0.0


def test_split_k_is_deterministic_and_equal_to_unsplit_sum():
    # 2 x 1 tiles with K = 32768: the reduction is split; two runs give the same bits
    T, n_out, n_in = 32768, 256, 256
    g = workloads.gradient((T, n_out), "student_t", seed=9, dtype="bf16")
    h = workloads.normal_bf16((T, n_in), seed=8)
    assert binding.mvue_gemm_workspace_bytes(0, n_out, n_in, T) > 0
    vals, meta = binding.mvue_prune(to_dev(g), 2, 4, 0, seed=2, layout=TC)
    a = binding.mvue_sparse_update_gemm(vals, meta, to_dev(h))
    b = binding.mvue_sparse_update_gemm(vals, meta, to_dev(h))
    assert torch.equal(a, b)
    v_ref, m_ref = oracle.prune(g, 2, 4, axis=0, seed=2, threads=oracle.host_threads())
    want = oracle.gemm(oracle.unpack(v_ref, m_ref), h, threads=oracle.host_threads())
    assert rel_fro(a.double().cpu().numpy(), want) <= TIGHT


def test_more_tiles_than_resident_pairs():
    # 8 x 12 = 96 output tiles for at most 74 resident pairs: every pair walks several tiles, the drained tile of
    # one overlapping the main loop of the next.  fp32 out, fp32 accumulate, and the same shape again must match.
    T, n_out, n_in = 512, 2048, 3072
    g = workloads.gradient((T, n_out), "student_t", seed=21, dtype="bf16")
    h = workloads.normal_bf16((T, n_in), seed=22)
    vals, meta = binding.mvue_prune(to_dev(g), 2, 4, 0, seed=5, layout=TC)
    assert binding.mvue_gemm_workspace_bytes(0, n_out, n_in, T) == 0
    a = binding.mvue_sparse_update_gemm(vals, meta, to_dev(h))
    b = binding.mvue_sparse_update_gemm(vals, meta, to_dev(h))
    assert torch.equal(a, b)
    acc = torch.full((n_out, n_in), -2.0, dtype=torch.float32, device="cuda")
    binding.mvue_sparse_update_gemm(vals, meta, to_dev(h), out=acc, accumulate=True)
    assert torch.allclose(acc, a - 2.0, rtol=1e-6, atol=1e-6)
    v_ref, m_ref = oracle.prune(g, 2, 4, axis=0, seed=5, threads=oracle.host_threads())
    want = oracle.gemm(oracle.unpack(v_ref, m_ref), h, threads=oracle.host_threads())
    assert rel_fro(a.double().cpu().numpy(), want) <= TIGHT
    # ragged edges in both directions with several rounds: 2056 x 3080 leaves 8-wide slivers of tiles
    g2 = workloads.gradient((T, n_out + 8), "student_t", seed=23, dtype="bf16")
    h2 = workloads.normal_bf16((T, n_in + 8), seed=24)
    vals2, meta2 = binding.mvue_prune(to_dev(g2), 2, 4, 0, seed=6, layout=TC)
    c = binding.mvue_sparse_update_gemm(vals2, meta2, to_dev(h2), out_dtype=torch.bfloat16)
    v_ref, m_ref = oracle.prune(g2, 2, 4, axis=0, seed=6, threads=oracle.host_threads())
    want2 = oracle.gemm(oracle.unpack(v_ref, m_ref), h2, threads=oracle.host_threads())
    assert rel_fro(c.double().cpu().numpy(), want2) <= 4e-3


def test_last_round_tiles_are_split_along_k():
    # 10 x 8 = 80 tiles over at most 74 resident pairs: the 6 tiles of the last round are cut along K into parts
    # (fp32 partial tiles in the workspace, summed by a second pass).  Rows from every row tile against the oracle;
    # the same bits when repeated; accumulate; and the whole-tile path (no workspace) agrees to rounding.
    T, n_out, n_in = 2048, 2560, 2048
    g = workloads.gradient((T, n_out), "student_t", seed=31, dtype="bf16")
    h = workloads.normal_bf16((T, n_in), seed=32)
    vals, meta = binding.mvue_prune(to_dev(g), 2, 4, 0, seed=8, layout=TC)
    need = binding.mvue_gemm_workspace_bytes(0, n_out, n_in, T)
    assert need > 0                                        # the tail split asks for room
    a = binding.mvue_sparse_update_gemm(vals, meta, to_dev(h))
    b = binding.mvue_sparse_update_gemm(vals, meta, to_dev(h))
    assert torch.equal(a, b)
    acc = torch.full((n_out, n_in), 0.25, dtype=torch.float32, device="cuda")
    binding.mvue_sparse_update_gemm(vals, meta, to_dev(h), out=acc, accumulate=True)
    assert torch.allclose(acc, a + 0.25, rtol=1e-6, atol=1e-6)
    # without a workspace the tiles stay whole (the raw entry point accepts NULL here)
    whole = torch.empty_like(a)
    L = binding.lib()
    hd = to_dev(h)
    rc = L.mvue_sparse_update_gemm(vals.data_ptr(), meta.data_ptr(), TC, n_out, T, hd.data_ptr(), n_in, n_in,
                                   whole.data_ptr(), 0, n_in, 0, None, 0, None, None)
    assert rc == 0
    torch.cuda.synchronize()
    assert torch.allclose(whole, a, rtol=1e-5, atol=1e-5)
    v_ref, m_ref = oracle.prune(g, 2, 4, axis=0, seed=8, threads=oracle.host_threads())
    rows = np.array(sorted({r for t in range(10) for r in (256 * t, 256 * t + 77, 256 * t + 130, 256 * t + 255)}))
    A_rows = np.ascontiguousarray(oracle.unpack(np.ascontiguousarray(v_ref[rows]), np.ascontiguousarray(m_ref[rows])))
    want = oracle.gemm(A_rows, h, threads=oracle.host_threads())
    got = a[torch.from_numpy(rows).cuda()].double().cpu().numpy()
    assert rel_fro(got, want) <= TIGHT
    assert np.abs(got - want).max() <= 1e-4 * np.abs(want).max()


def test_gemm_argument_checks():
    vals = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    meta = torch.zeros((64, 16), dtype=torch.uint8, device="cuda")
    h = torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda")
    L = binding.lib()
    # K = 192 is not a multiple of 128
    assert L.mvue_sparse_update_gemm(vals.data_ptr(), meta.data_ptr(), TC, 64, 192, h.data_ptr(), 64, 64,
                                     h.data_ptr(), 0, 64, 0, None, 0, None, None) == -3
    assert L.mvue_sparse_update_gemm(None, meta.data_ptr(), TC, 64, 128, h.data_ptr(), 64, 64,
                                     h.data_ptr(), 0, 64, 0, None, 0, None, None) == -1
    # the products read the tensor-core metadata order only
    assert L.mvue_sparse_update_gemm(vals.data_ptr(), meta.data_ptr(), 0, 64, 128, h.data_ptr(), 64, 64,
                                     h.data_ptr(), 0, 64, 0, None, 0, None, None) == -6
    # accumulate into bf16 is refused
    assert L.mvue_sparse_update_gemm(vals.data_ptr(), meta.data_ptr(), TC, 64, 128, h.data_ptr(), 64, 64,
                                     h.data_ptr(), 1, 64, 1, None, 0, None, None) == -5
    # a reduction that needs split-K refuses a missing workspace
    big_k = 1 << 16
    if binding.mvue_gemm_workspace_bytes(0, 64, 64, big_k) > 0:
        assert L.mvue_sparse_update_gemm(vals.data_ptr(), meta.data_ptr(), TC, 64, big_k, h.data_ptr(), 64, 64,
                                         h.data_ptr(), 0, 64, 0, None, 0, None, None) == -7


def test_issue_rate_probe_runs_and_counts_its_work():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pairs, flops = binding.mvue_probe_sparse_mma(256, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and pairs >= 1
    assert flops == pairs * 256 * 4 * 2.0 * 256 * 256 * 32
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    binding.mvue_probe_sparse_mma(2048, status)
    e1.record()
    torch.cuda.synchronize()
    # back-to-back sparse MMAs on resident operands must beat the dense bf16 rate any library reaches on this part
    assert pairs * 2048 * 4 * 2.0 * 256 * 256 * 32 / (e0.elapsed_time(e1) * 1e-3) > 2.0e15
    for bad in (0, -1, (1 << 20) + 1):
        with pytest.raises(binding.MvueError) as e:
            binding.mvue_probe_sparse_mma(bad)
        assert e.value.status == -3


def test_long_reduction_ragged_output_with_and_without_the_tail_split():
    # K = 16384 (128 stages per tile): the small-footprint fp32 epilogue.  9 x 10 = 90 ragged tiles (2056 x 2312: 8-wide
    # slivers in both directions) over at most 74 resident pairs: with the workspace the last round's tiles are cut
    # along K (partial tiles written by the same epilogue), without it they stay whole; accumulate; sampled rows of
    # every row tile, the sliver included, against the oracle.
    T, n_out, n_in = 16384, 2056, 2312
    g = workloads.gradient((T, n_out), "student_t", seed=41, dtype="bf16")
    h = workloads.normal_bf16((T, n_in), seed=42)
    gd, hd = to_dev(g), to_dev(h)
    vals, meta = binding.mvue_prune(gd, 2, 4, 0, seed=9, layout=TC)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    a = binding.mvue_sparse_update_gemm(vals, meta, hd, dev_status=st)            # workspace from the binding
    whole = torch.empty_like(a)
    rc = binding.lib().mvue_sparse_update_gemm(vals.data_ptr(), meta.data_ptr(), TC, n_out, T, hd.data_ptr(), n_in, n_in,
                                               whole.data_ptr(), 0, n_in, 0, None, 0, st.data_ptr(), None)
    assert rc == 0
    acc = torch.full((n_out, n_in), 1.5, dtype=torch.float32, device="cuda")
    binding.mvue_sparse_update_gemm(vals, meta, hd, out=acc, accumulate=True)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    # the K parts are summed in another order than the whole tile: fp32 rounding of sums of ~0.3-sized entries
    assert float((whole - a).abs().max()) <= 1e-5 and rel_fro(whole.double().cpu().numpy(), a.double().cpu().numpy()) <= 1e-6
    assert torch.allclose(acc, a + 1.5, rtol=1e-6, atol=1e-6)
    v_ref, m_ref = oracle.prune(g, 2, 4, axis=0, seed=9, threads=oracle.host_threads())
    rows = np.array(sorted({min(r, n_out - 1) for t in range(9) for r in (256 * t, 256 * t + 131, 256 * t + 255)}))
    A_rows = np.ascontiguousarray(oracle.unpack(np.ascontiguousarray(v_ref[rows]), np.ascontiguousarray(m_ref[rows])))
    want = oracle.gemm(A_rows, h, threads=oracle.host_threads())
    for out in (a, whole):
        got = out[torch.from_numpy(rows).cuda()].double().cpu().numpy()
        assert rel_fro(got, want) <= TIGHT

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

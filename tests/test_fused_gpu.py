"""The fused prune -> update product against the oracle (prune, unpack, fp64 product) and against the
separate calls with the same seed."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_10991_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def to_dev(a):
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


# in = 8 .. 264: one or two column tiles (no cluster, clusters of two); 520: three tiles (no cluster); 1024, 2048 + 8:
# four tiles (clusters of four, the blocks share every pruned stage) and nine (no cluster); ragged rows and columns
@pytest.mark.parametrize("T,n_out,n_in", [(128, 8, 8), (512, 256, 256), (640, 136, 264), (4096, 384, 520),
                                          (16384, 128, 256), (1024, 264, 1024), (2048, 128, 2048), (512, 520, 2056)])
@pytest.mark.parametrize("n,m,joint", [(2, 4, 0), (2, 4, 1), (1, 2, 0)])
def test_fused_matches_oracle_and_separate_calls(T, n_out, n_in, n, m, joint):
    g = workloads.gradient((T, n_out), "relu_lognormal", seed=T + n_out, dtype="bf16")
    h = workloads.normal_bf16((T, n_in), seed=3)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    fused = binding.mvue_fused_update_gemm(to_dev(g), to_dev(h), n, m, seed=17, dev_status=st, joint=joint)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    v_ref, m_ref = oracle.prune(g, n, m, axis=0, seed=17, threads=oracle.host_threads(), joint=joint)
    want = oracle.gemm(oracle.unpack(v_ref, m_ref), h, threads=oracle.host_threads())
    err = np.linalg.norm(fused.double().cpu().numpy() - want) / max(np.linalg.norm(want), 1e-300)
    assert err <= 1e-2 and err <= 2e-5, err
    vals, meta = binding.mvue_prune(to_dev(g), n, m, 0, seed=17, layout=binding.MVUE_LAYOUT_TC, joint=joint)
    sep = binding.mvue_sparse_update_gemm(vals, meta, to_dev(h))
    assert torch.allclose(fused, sep, rtol=1e-5, atol=1e-6 * float(sep.abs().max()))


def test_fused_argument_checks():
    g = torch.zeros((128, 64), dtype=torch.float32, device="cuda")
    h = torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.MvueError) as e:
        binding.mvue_fused_update_gemm(g, h, 2, 4, 0)           # fp32 gradients are not taken by the fused path
    assert e.value.status == -5
    with pytest.raises(binding.MvueError) as e:
        binding.mvue_fused_update_gemm(h, h, 1, 4, 0)
    assert e.value.status == -2

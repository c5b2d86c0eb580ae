"""mvue_sparse_backward_gemm_pruned: the backward product whose epilogue prunes its own bf16 output along the next
product's reduction axis.  Everything it writes must equal, bit for bit, what the separate calls write: the backward
product, then mvue_prune of the stored result (both checked against the oracle elsewhere)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2203_10991_b200 import binding, workloads
from tests.helpers import layouts

pytestmark = pytest.mark.gpu
TC = binding.MVUE_LAYOUT_TC


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


# (T, out, in): one launch with the prune in the epilogue (enough tiles, T a multiple of 128), a ragged last column
# tile, and two shapes that take the two-step route (a product split along K; a ragged last row block)
SHAPES = [(4096, 512, 2048), (2048, 1024, 2432), (512, 1024, 256), (4096 + 64, 512, 2048)]


@pytest.mark.parametrize("T,n_out,n_in", SHAPES)
@pytest.mark.parametrize("joint", [binding.MVUE_JOINT_SYSTEMATIC, binding.MVUE_JOINT_TABLE])
@pytest.mark.parametrize("options", [binding.MVUE_OPT_NONE, binding.MVUE_OPT_EPS16,
                                     binding.MVUE_OPT_EPS16 | binding.MVUE_OPT_STOCHASTIC_ROUNDING])
def test_equals_the_separate_calls_bit_for_bit(T, n_out, n_in, joint, options):
    eps16 = bool(options & binding.MVUE_OPT_EPS16)
    sr = bool(options & binding.MVUE_OPT_STOCHASTIC_ROUNDING)        # (takes the two-step route inside the entry point)
    g = to_dev(workloads.gradient((T, n_out), "student_t", seed=T + n_in, dtype="bf16"))
    W = to_dev(workloads.normal_bf16((n_out, n_in), seed=3, std=n_out ** -0.5))
    fz = to_dev(workloads.normal_bf16((T, n_in), seed=4))
    vals, meta = binding.mvue_prune(g, 2, 4, 1, seed=11, layout=TC, joint=joint)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dh, nv, nm = binding.mvue_sparse_backward_gemm_pruned(vals, meta, W, fz, next_seed=12, next_joint=joint,
                                                          next_options=options, dev_status=status)
    want_dh = binding.mvue_sparse_backward_gemm(vals, meta, W, act_grad=fz, out_dtype=torch.bfloat16, dev_status=status)
    want_v, want_m = binding.mvue_prune(want_dh, 2, 4, 1, seed=12, layout=TC, joint=joint, options=options)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(dh.view(torch.int16), want_dh.view(torch.int16))
    assert torch.equal(nv.view(torch.int16), want_v.view(torch.int16))
    assert torch.equal(nm.reshape(-1), want_m.reshape(-1))
    # and against the oracle's prune of the stored product (sampled rows: any row is computable on its own)
    dh_np = dh.view(torch.int16).cpu().numpy().view(np.uint16)
    rows = sorted({0, 127, 128, T - 1, T // 2 + 5})
    nv_np = nv.view(torch.int16).cpu().numpy().view(np.uint16)
    for i, r in enumerate(rows):
        # row r of the operand draws the words of row r: re-run the oracle with the row's global block numbers
        v1, m1 = oracle.prune(np.ascontiguousarray(dh_np[r:r + 1]), 2, 4, axis=1, seed=12, joint=joint,
                              k_total=n_in * (r + 1), k_offset=n_in * r, eps16=eps16, stochastic_rounding=sr)
        assert np.array_equal(nv_np[r], v1[0]), r
    nm_canon = layouts.tc_to_canonical(nm.cpu().numpy().reshape(-1), T, n_in)
    for r in rows:
        _, m1 = oracle.prune(np.ascontiguousarray(dh_np[r:r + 1]), 2, 4, axis=1, seed=12, joint=joint,
                             k_total=n_in * (r + 1), k_offset=n_in * r, eps16=eps16)
        assert np.array_equal(nm_canon[r], m1[0]), r


def test_arguments():
    T, n_out, n_in = 256, 256, 192                                  # in is not a multiple of 128
    g = to_dev(workloads.gradient((T, n_out), "student_t", seed=1, dtype="bf16"))
    W = to_dev(workloads.normal_bf16((n_out, n_in), seed=3))
    fz = to_dev(workloads.normal_bf16((T, n_in), seed=4))
    vals, meta = binding.mvue_prune(g, 2, 4, 1, seed=11, layout=TC)
    L = binding.lib()
    rc = L.mvue_sparse_backward_gemm_pruned(vals.data_ptr(), meta.data_ptr(), TC, T, n_out, W.data_ptr(), n_in, n_in,
                                            fz.data_ptr(), fz.data_ptr(), n_in, 0, 0, 0, fz.data_ptr(), fz.data_ptr(), None, 0,
                                            None, None)
    assert rc == -3
    rc = L.mvue_sparse_backward_gemm_pruned(vals.data_ptr(), meta.data_ptr(), TC, T, n_out, W.data_ptr(), n_in, n_in,
                                            None, fz.data_ptr(), n_in, 0, 0, 0, fz.data_ptr(), fz.data_ptr(), None, 0, None, None)
    assert rc == -1
    rc = L.mvue_sparse_backward_gemm_pruned(vals.data_ptr(), meta.data_ptr(), TC, T, n_out, W.data_ptr(), n_in, n_in,
                                            fz.data_ptr(), fz.data_ptr(), n_in, 0, 0, 4, fz.data_ptr(), fz.data_ptr(), None, 0,
                                            None, None)
    assert rc == -12                                                # an option bit the library does not know

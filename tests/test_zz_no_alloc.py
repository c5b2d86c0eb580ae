"""mvue_sparse_update_gemm_noalloc: the update product for callers that cannot allocate device memory
(a plugin whose host owns the allocator, a loop in which allocation is forbidden after start-up).
Its split-K scratch is a fixed array inside the library, so the entry point must give the same
numbers as mvue_sparse_update_gemm with a caller-supplied workspace -- on a first call, and again
on a second call that finds the first call's leftovers in the shared array.

This file is named to be collected last: if it fails, a run that stops at the first failure has
already run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2203_10991_b200 import binding, workloads

pytestmark = pytest.mark.gpu
TC = binding.MVUE_LAYOUT_TC


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # small output, long reduction: the product is split along K and really uses the scratch
    T, n_out, n_in = 4096, 256, 256
    assert 0 < binding.mvue_gemm_workspace_bytes(0, n_out, n_in, T) <= (8 << 20)
    h = to_dev(workloads.normal_bf16((T, n_in), seed=12))
    outs = []
    for call, seed in enumerate((3, 4)):          # second call: other data, same shared scratch
        g = workloads.gradient((T, n_out), "student_t", seed=seed, dtype="bf16")
        vals, meta = binding.mvue_prune(to_dev(g), 2, 4, 0, seed=seed, layout=TC)
        want = binding.mvue_sparse_update_gemm(vals, meta, h)
        got = torch.empty_like(want)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        binding.mvue_sparse_update_gemm_noalloc(vals, meta, h, got, dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # same kernels, same split, same summation order: the tolerance of the GEMM tests is met
        # with room to spare (the results are in fact identical)
        err = float((got.double() - want.double()).norm() / want.double().norm())
        assert err <= 2e-5, (call, err)
        outs.append(got)
    assert not torch.equal(outs[0], outs[1])      # the two calls did compute different products
    # accumulate works through the same path
    acc = outs[1].clone()
    binding.mvue_sparse_update_gemm_noalloc(vals, meta, h, acc, accumulate=True)
    assert torch.allclose(acc, 2 * outs[1], rtol=1e-6, atol=1e-7)


def test_sizes_beyond_the_library_scratch_are_refused():
    # a 256 x 2304 output over 200704 rows is split eight ways on a 148-SM part: 18 MiB of partial sums
    n_out, n_in, T = 256, 2304, 200704
    need = binding.mvue_gemm_workspace_bytes(0, n_out, n_in, T)
    if need <= (8 << 20):
        pytest.skip("this device splits the problem less than expected")
    fake = ctypes.c_void_p(1 << 20)
    rc = binding.lib().mvue_sparse_update_gemm_noalloc(fake, fake, TC, n_out, T, fake, n_in, n_in, fake, 0, n_in,
                                                       0, None, None)
    assert rc == -7

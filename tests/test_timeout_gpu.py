"""The bounded-wait exit of the product kernels, exercised without a fault: the self-test launch waits on a
barrier that nobody arrives on (nothing is issued, nothing is in flight), the wait gives up after a few thousand
polls, MVUE_ERR_DEVICE_TIMEOUT lands in the status word, the blocks meet at their cluster barrier and hand
tensor memory back.  Afterwards the context is healthy: the same product gives the same bits as before."""
import numpy as np
import pytest
import torch

from paper_2203_10991_b200 import binding, workloads

pytestmark = pytest.mark.gpu
TC = binding.MVUE_LAYOUT_TC
MVUE_ERR_DEVICE_TIMEOUT = -10


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def test_an_unanswered_wait_expires_and_reports_timeout():
    T, n_out, n_in = 1024, 512, 512
    g = to_dev(workloads.gradient((T, n_out), "student_t", seed=21, dtype="bf16"))
    h = to_dev(workloads.normal_bf16((T, n_in), seed=22))
    vals, meta = binding.mvue_prune(g, 2, 4, 0, seed=5, layout=TC)
    ok_status = torch.zeros(1, dtype=torch.int32, device="cuda")
    before = binding.mvue_sparse_update_gemm(vals, meta, h, dev_status=ok_status).clone()
    torch.cuda.synchronize()
    assert int(ok_status.item()) == 0

    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for polls in (200, 3000):                        # below and above where the poll loop starts to sleep
        status.zero_()
        binding.mvue_selftest_wait_timeout(polls, status)
        torch.cuda.synchronize()                     # the launch ends by itself
        assert int(status.item()) == MVUE_ERR_DEVICE_TIMEOUT

    # tensor memory came back and nothing is wedged: the issue-rate probe (which allocates all of it on every SM)
    # completes, and the product is bit-identical to the run before the timeouts
    probe_status = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.mvue_probe_sparse_mma(16, probe_status)
    after = binding.mvue_sparse_update_gemm(vals, meta, h, dev_status=ok_status)
    torch.cuda.synchronize()
    assert int(probe_status.item()) == 0 and int(ok_status.item()) == 0
    assert torch.equal(before, after)

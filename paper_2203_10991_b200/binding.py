"""Python binding of the C ABI in include/mvue.h: argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory; every function passes
raw pointers, sizes and the current CUDA stream to the library.  There is no
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libmvue_b200.so"
_lib = None

MVUE_F32, MVUE_BF16 = 0, 1
MVUE_LAYOUT_CANONICAL = 0
MVUE_LAYOUT_TC = 1
MVUE_JOINT_TABLE, MVUE_JOINT_SYSTEMATIC, MVUE_JOINT_APPROX = 0, 1, 2
MVUE_OPT_NONE, MVUE_OPT_STOCHASTIC_ROUNDING, MVUE_OPT_EPS16 = 0, 1, 2

EXPORTS = ("mvue_version", "mvue_status_string", "mvue_last_cuda_error", "mvue_packed_sizes",
           "mvue_prune", "mvue_prune_joint", "mvue_prune_opts", "mvue_prune_4of8", "mvue_unpack", "mvue_sparse_update_gemm", "mvue_sparse_backward_gemm",
           "mvue_sparse_backward_gemm_pruned",
           "mvue_gemm_workspace_bytes", "mvue_sparse_update_gemm_noalloc", "mvue_fused_update_gemm", "mvue_fused_update_gemm_joint",
           "mvue_probe_sparse_mma", "mvue_selftest_wait_timeout")


class MvueError(RuntimeError):
    def __init__(self, status: int, what: str):
        L = lib()
        msg = L.mvue_status_string(status).decode()
        cuda = L.mvue_last_cuda_error().decode()
        super().__init__(f"{what}: {msg} [{status}]" + (f" -- {cuda}" if status == -9 and cuda else ""))
        self.status = status


def lib() -> ctypes.CDLL:
    """Load libmvue_b200.so (built by `python -m paper_2203_10991_b200.build`)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                               "`python -m paper_2203_10991_b200.build` (there is no CPU fallback)")
        L = ctypes.CDLL(str(_LIB_PATH))
        i64, u64, vp, ci = ctypes.c_int64, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int
        szp = ctypes.POINTER(ctypes.c_size_t)
        L.mvue_version.restype = ci
        L.mvue_status_string.argtypes = [ci]
        L.mvue_status_string.restype = ctypes.c_char_p
        L.mvue_last_cuda_error.restype = ctypes.c_char_p
        L.mvue_packed_sizes.argtypes = [i64, i64, ci, ci, ci, ci, szp, szp]
        L.mvue_prune.argtypes = [vp, ci, i64, i64, i64, ci, ci, ci, u64, i64, i64, vp, vp, ci, vp]
        L.mvue_prune_joint.argtypes = [vp, ci, i64, i64, i64, ci, ci, ci, u64, i64, i64, vp, vp, ci, ci, vp]
        L.mvue_prune_opts.argtypes = [vp, ci, i64, i64, i64, ci, ci, ci, u64, i64, i64, vp, vp, ci, ci, ctypes.c_uint, vp]
        L.mvue_prune_4of8.argtypes = [vp, ci, i64, i64, i64, ci, u64, i64, i64, vp, vp, vp]
        L.mvue_unpack.argtypes = [vp, vp, ci, i64, i64, vp, vp]
        L.mvue_sparse_update_gemm.argtypes = [vp, vp, ci, i64, i64, vp, i64, i64, vp, ci, i64, ci, vp,
                                              ctypes.c_size_t, vp, vp]
        L.mvue_sparse_backward_gemm.argtypes = [vp, vp, ci, i64, i64, vp, i64, i64, vp, vp, ci, i64, vp,
                                                ctypes.c_size_t, vp, vp]
        L.mvue_sparse_backward_gemm_pruned.argtypes = [vp, vp, ci, i64, i64, vp, i64, i64, vp, vp, i64, u64, ci,
                                                       ctypes.c_uint, vp, vp, vp, ctypes.c_size_t, vp, vp]
        L.mvue_gemm_workspace_bytes.argtypes = [ci, i64, i64, i64, szp]
        L.mvue_fused_update_gemm.argtypes = [vp, ci, i64, i64, i64, ci, ci, u64, vp, i64, i64, vp, ci, i64, ci, vp,
                                             ctypes.c_size_t, vp, vp]
        L.mvue_fused_update_gemm_joint.argtypes = [vp, ci, i64, i64, i64, ci, ci, ci, u64, vp, i64, i64, vp, ci, i64, ci, vp,
                                                   ctypes.c_size_t, vp, vp]
        L.mvue_sparse_update_gemm_noalloc.argtypes = [vp, vp, ci, i64, i64, vp, i64, i64, vp, ci, i64, ci, vp, vp]
        L.mvue_probe_sparse_mma.argtypes = [ci, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_double), vp, vp]
        L.mvue_selftest_wait_timeout.argtypes = [ci, vp, vp]
        _lib = L
    return _lib


def _check(status: int, what: str):
    if status != 0:
        raise MvueError(status, what)


def _stream_ptr() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return MVUE_F32
    if t.dtype == torch.bfloat16:
        return MVUE_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def mvue_packed_sizes(rows: int, cols: int, n: int, m: int, axis: int, layout: int = MVUE_LAYOUT_CANONICAL):
    vb, mb = ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().mvue_packed_sizes(rows, cols, n, m, axis, layout, ctypes.byref(vb), ctypes.byref(mb)),
           "mvue_packed_sizes")
    return vb.value, mb.value


def mvue_prune(g: torch.Tensor, n: int, m: int, axis: int, seed: int, *, k_total: int | None = None,
               k_offset: int = 0, values: torch.Tensor | None = None, meta: torch.Tensor | None = None,
               layout: int = MVUE_LAYOUT_CANONICAL, joint: int | None = None, options: int = MVUE_OPT_NONE):
    """MVUE n:m prune + pack of a 2-D CUDA tensor g (fp32 or bf16, unit column stride).

    joint: None calls mvue_prune (App. A.2 pair table); an mvue_joint value calls mvue_prune_joint.
    options: non-zero calls mvue_prune_opts (MVUE_OPT_STOCHASTIC_ROUNDING: unbiased bf16 storage of the survivors).
    Returns (values bf16 [Mrows, K/2], meta uint8 [Mrows, K/8]).
    """
    assert g.is_cuda and g.dim() == 2 and g.stride(1) == 1
    rows, cols = g.shape
    mrows, k = (rows, cols) if axis == 1 else (cols, rows)
    if values is None or meta is None:
        _, meta_bytes = mvue_packed_sizes(rows, cols, n, m, axis, layout)   # validates before allocating
        values = torch.empty((mrows, k // 2), dtype=torch.bfloat16, device=g.device)
        meta = torch.empty((meta_bytes // (k // 8), k // 8), dtype=torch.uint8, device=g.device)
    if options:
        _check(lib().mvue_prune_opts(g.data_ptr(), _dtype_code(g), rows, cols, g.stride(0), n, m, axis,
                                     seed & (2**64 - 1), k if k_total is None else k_total, k_offset,
                                     values.data_ptr(), meta.data_ptr(), layout,
                                     MVUE_JOINT_TABLE if joint is None else int(joint), int(options), _stream_ptr()),
               "mvue_prune_opts")
    elif joint is None:
        _check(lib().mvue_prune(g.data_ptr(), _dtype_code(g), rows, cols, g.stride(0), n, m, axis,
                                seed & (2**64 - 1), k if k_total is None else k_total, k_offset,
                                values.data_ptr(), meta.data_ptr(), layout, _stream_ptr()), "mvue_prune")
    else:
        _check(lib().mvue_prune_joint(g.data_ptr(), _dtype_code(g), rows, cols, g.stride(0), n, m, axis,
                                      seed & (2**64 - 1), k if k_total is None else k_total, k_offset,
                                      values.data_ptr(), meta.data_ptr(), layout, int(joint), _stream_ptr()),
               "mvue_prune_joint")
    return values, meta


def mvue_prune_4of8(g: torch.Tensor, axis: int, seed: int, *, k_total: int | None = None, k_offset: int = 0):
    """Approx-4:8 prune (prune only) of a 2-D CUDA tensor: (values bf16 [Mrows, K/2], mask uint8 [Mrows, K/8])."""
    assert g.is_cuda and g.dim() == 2 and g.stride(1) == 1
    rows, cols = g.shape
    mrows, k = (rows, cols) if axis == 1 else (cols, rows)
    values = torch.empty((mrows, k // 2), dtype=torch.bfloat16, device=g.device)
    mask = torch.empty((mrows, k // 8), dtype=torch.uint8, device=g.device)
    _check(lib().mvue_prune_4of8(g.data_ptr(), _dtype_code(g), rows, cols, g.stride(0), axis, seed & (2**64 - 1),
                                 k if k_total is None else k_total, k_offset, values.data_ptr(), mask.data_ptr(),
                                 _stream_ptr()), "mvue_prune_4of8")
    return values, mask


def mvue_unpack(values: torch.Tensor, meta: torch.Tensor, layout: int = MVUE_LAYOUT_CANONICAL) -> torch.Tensor:
    mrows, kh = values.shape
    dense = torch.empty((mrows, 2 * kh), dtype=torch.bfloat16, device=values.device)
    _check(lib().mvue_unpack(values.data_ptr(), meta.data_ptr(), layout, mrows, 2 * kh, dense.data_ptr(),
                             _stream_ptr()), "mvue_unpack")
    return dense


def mvue_gemm_workspace_bytes(which: int, M: int, N: int, K: int) -> int:
    b = ctypes.c_size_t()
    _check(lib().mvue_gemm_workspace_bytes(which, M, N, K, ctypes.byref(b)), "mvue_gemm_workspace_bytes")
    return b.value


def _workspace(which, M, N, K, device, workspace):
    need = mvue_gemm_workspace_bytes(which, M, N, K)
    if need == 0:
        return None, 0
    if workspace is None or workspace.numel() * workspace.element_size() < need:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace, workspace.numel() * workspace.element_size()


def mvue_sparse_update_gemm(values: torch.Tensor, meta: torch.Tensor, h: torch.Tensor, *,
                            out: torch.Tensor | None = None, out_dtype=torch.float32, accumulate: bool = False,
                            workspace: torch.Tensor | None = None, dev_status: torch.Tensor | None = None,
                            layout: int = MVUE_LAYOUT_TC) -> torch.Tensor:
    """dW[out, in] (+)= theta(g)^T . h with the packed operand of mvue_prune(g, axis=0, layout=MVUE_LAYOUT_TC)."""
    n_out, half_t = values.shape
    T, n_in = h.shape
    assert h.dtype == torch.bfloat16 and h.stride(1) == 1 and 2 * half_t == T
    if out is None:
        out = torch.empty((n_out, n_in), dtype=out_dtype, device=h.device)
    ws, ws_bytes = _workspace(0, n_out, n_in, T, h.device, workspace)
    _check(lib().mvue_sparse_update_gemm(values.data_ptr(), meta.data_ptr(), layout, n_out, T, h.data_ptr(), n_in,
                                         h.stride(0), out.data_ptr(), _dtype_code(out), out.stride(0),
                                         int(accumulate), None if ws is None else ws.data_ptr(), ws_bytes,
                                         None if dev_status is None else dev_status.data_ptr(), _stream_ptr()),
           "mvue_sparse_update_gemm")
    return out


def mvue_sparse_backward_gemm(values: torch.Tensor, meta: torch.Tensor, W: torch.Tensor, *,
                              act_grad: torch.Tensor | None = None, out: torch.Tensor | None = None,
                              out_dtype=torch.bfloat16, workspace: torch.Tensor | None = None,
                              dev_status: torch.Tensor | None = None,
                              layout: int = MVUE_LAYOUT_TC) -> torch.Tensor:
    """dh[T, in] = (theta(g) . W) (* act_grad) with the packed operand of mvue_prune(g, axis=1, layout=MVUE_LAYOUT_TC)."""
    T, half_o = values.shape
    n_out, n_in = W.shape
    assert W.dtype == torch.bfloat16 and W.stride(1) == 1 and 2 * half_o == n_out
    if out is None:
        out = torch.empty((T, n_in), dtype=out_dtype, device=W.device)
    if act_grad is not None:
        assert act_grad.dtype == torch.bfloat16 and act_grad.shape == out.shape and act_grad.stride(0) == out.stride(0)
    ws, ws_bytes = _workspace(1, T, n_in, n_out, W.device, workspace)
    _check(lib().mvue_sparse_backward_gemm(values.data_ptr(), meta.data_ptr(), layout, T, n_out, W.data_ptr(), n_in,
                                           W.stride(0), None if act_grad is None else act_grad.data_ptr(),
                                           out.data_ptr(), _dtype_code(out), out.stride(0),
                                           None if ws is None else ws.data_ptr(), ws_bytes,
                                           None if dev_status is None else dev_status.data_ptr(), _stream_ptr()),
           "mvue_sparse_backward_gemm")
    return out


def mvue_sparse_backward_gemm_pruned(values: torch.Tensor, meta: torch.Tensor, W: torch.Tensor, act_grad: torch.Tensor,
                                     next_seed: int, *, next_joint: int = MVUE_JOINT_TABLE, next_options: int = MVUE_OPT_NONE,
                                     workspace: torch.Tensor | None = None, dev_status: torch.Tensor | None = None,
                                     layout: int = MVUE_LAYOUT_TC):
    """dh = (theta(g) . W) * act_grad (bf16) and, from the same launch, dh pruned 2:4 along its columns in tensor-core
    order (what mvue_prune(dh, 2, 4, axis=1, next_seed, layout=MVUE_LAYOUT_TC, joint=next_joint,
    options=next_options) gives).
    Returns (dh, next_values, next_meta)."""
    T, half_o = values.shape
    n_out, n_in = W.shape
    assert W.dtype == torch.bfloat16 and W.stride(1) == 1 and 2 * half_o == n_out
    out = torch.empty((T, n_in), dtype=torch.bfloat16, device=W.device)
    assert act_grad.dtype == torch.bfloat16 and act_grad.shape == out.shape and act_grad.stride(0) == out.stride(0)
    _, meta_bytes = mvue_packed_sizes(T, n_in, 2, 4, 1, MVUE_LAYOUT_TC)
    next_values = torch.empty((T, n_in // 2), dtype=torch.bfloat16, device=W.device)
    next_meta = torch.empty((meta_bytes // (n_in // 8), n_in // 8), dtype=torch.uint8, device=W.device)
    ws, ws_bytes = _workspace(1, T, n_in, n_out, W.device, workspace)
    _check(lib().mvue_sparse_backward_gemm_pruned(values.data_ptr(), meta.data_ptr(), layout, T, n_out, W.data_ptr(), n_in,
                                                  W.stride(0), act_grad.data_ptr(), out.data_ptr(), out.stride(0),
                                                  next_seed & (2**64 - 1), int(next_joint), int(next_options), next_values.data_ptr(),
                                                  next_meta.data_ptr(), None if ws is None else ws.data_ptr(), ws_bytes,
                                                  None if dev_status is None else dev_status.data_ptr(), _stream_ptr()),
           "mvue_sparse_backward_gemm_pruned")
    return out, next_values, next_meta


def mvue_sparse_update_gemm_noalloc(values: torch.Tensor, meta: torch.Tensor, h: torch.Tensor, out: torch.Tensor, *,
                                    accumulate: bool = False, dev_status: torch.Tensor | None = None,
                                    layout: int = MVUE_LAYOUT_TC) -> torch.Tensor:
    """The update product for callers that may not allocate: the caller passes every buffer, including
    `out`, and the split-K scratch is the fixed array inside the library (8 MiB per GPU).  Nothing is
    allocated here either.  Raises MvueError(-7) when the problem needs more scratch than that."""
    n_out, half_t = values.shape
    T, n_in = h.shape
    _check(lib().mvue_sparse_update_gemm_noalloc(values.data_ptr(), meta.data_ptr(), layout, n_out, T, h.data_ptr(),
                                                 n_in, h.stride(0), out.data_ptr(), _dtype_code(out), out.stride(0),
                                                 int(accumulate),
                                                 None if dev_status is None else dev_status.data_ptr(),
                                                 _stream_ptr()), "mvue_sparse_update_gemm_noalloc")
    return out


def mvue_fused_update_gemm(g: torch.Tensor, h: torch.Tensor, n: int, m: int, seed: int, *,
                           out: torch.Tensor | None = None, out_dtype=torch.float32, accumulate: bool = False,
                           workspace: torch.Tensor | None = None,
                           dev_status: torch.Tensor | None = None, joint: int = MVUE_JOINT_TABLE) -> torch.Tensor:
    """dW[out, in] (+)= theta(g)^T . h in one kernel: g bf16 [T, out] is pruned along the tokens on the fly
    (joint: the 2:4 law, MVUE_JOINT_TABLE or MVUE_JOINT_SYSTEMATIC)."""
    T, n_out = g.shape
    T2, n_in = h.shape
    assert T == T2 and g.stride(1) == 1 and h.stride(1) == 1
    if out is None:
        out = torch.empty((n_out, n_in), dtype=out_dtype, device=h.device)
    ws, ws_bytes = _workspace(2, n_out, n_in, T, h.device, workspace)
    _check(lib().mvue_fused_update_gemm_joint(g.data_ptr(), _dtype_code(g), T, n_out, g.stride(0), n, m, int(joint),
                                              seed & (2**64 - 1),
                                        h.data_ptr(), n_in, h.stride(0), out.data_ptr(), _dtype_code(out),
                                        out.stride(0), int(accumulate), None if ws is None else ws.data_ptr(), ws_bytes,
                                        None if dev_status is None else dev_status.data_ptr(), _stream_ptr()),
           "mvue_fused_update_gemm")
    return out


def mvue_probe_sparse_mma(iters: int, dev_status: torch.Tensor | None = None):
    """One launch of the sparse tensor-core issue-rate probe on the current stream.
    Returns (pairs, dense-equivalent flops of the launch); time it with CUDA events."""
    pairs, flops = ctypes.c_int(), ctypes.c_double()
    _check(lib().mvue_probe_sparse_mma(iters, ctypes.byref(pairs), ctypes.byref(flops),
                                       None if dev_status is None else dev_status.data_ptr(), _stream_ptr()),
           "mvue_probe_sparse_mma")
    return pairs.value, flops.value


def mvue_selftest_wait_timeout(polls: int, dev_status: torch.Tensor) -> None:
    """One launch whose only wait nobody answers: it expires after `polls` polls and the blocks leave through the
    ordinary exit, writing MVUE_ERR_DEVICE_TIMEOUT (-10) to dev_status (int32 CUDA tensor)."""
    _check(lib().mvue_selftest_wait_timeout(polls, dev_status.data_ptr(), _stream_ptr()), "mvue_selftest_wait_timeout")

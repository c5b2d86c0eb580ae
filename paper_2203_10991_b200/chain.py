"""Backward + update pass of an MLP stack with every neural gradient MVUE-pruned.

For each linear layer l (top to bottom), with g = dC/dz_l [T x out], its input activations h [T x in], weights
W [out x in] and the derivative f'(z) of the activation below it:
    update:   dW_l = theta_0(g)^T h          (prune along tokens, sparse update product)
    backward: g_below = (theta_1(g) W) * f'(z_below)   (independent prune along out, sparse backward product)
Only calls into the C-ABI library; torch tensors are device memory.  The forward pass that produces h and f'(z)
is the caller's business.
"""
from __future__ import annotations

import torch

from . import binding

TC = binding.MVUE_LAYOUT_TC


def layer_seeds(base_seed: int, layer: int) -> tuple[int, int]:
    """Distinct seeds for the two prunes of one layer's gradient (update / backward)."""
    return (base_seed * 0x9E3779B97F4A7C15 + 2 * layer) & (2**64 - 1), \
           (base_seed * 0x9E3779B97F4A7C15 + 2 * layer + 1) & (2**64 - 1)


def backward_update(g_top: torch.Tensor, layers, n: int = 2, m: int = 4, base_seed: int = 0, joint: int | None = None,
                    overlap: bool = False, prune_in_epilogue_min_k: int | None = None, options: int = 0):
    """layers: list (top layer first) of dicts {"W": [out x in] bf16, "h": [T x in] bf16,
    "act_grad": [T x in] bf16 or None (None for the bottom layer: no gradient is propagated further)}.
    joint: the 2:4 law over pairs handed to mvue_prune_joint (None: mvue_prune, the App. A.2 table).
    overlap: run each layer's update product on a second stream beside the prune that feeds its backward product.
    The product issues on a few percent of an SM's instruction slots and the prune uses no tensor core; the update
    product of a long token axis keeps a small register footprint, so blocks of the (shared-memory-free) prune along
    the features fit on the same SMs.  Same calls, same seeds, same results; the streams join before each backward
    product and before returning.
    options: mvue_prune_option bits handed to every prune (stochastic rounding, sixteen random bits per block).
    prune_in_epilogue_min_k: when set (2:4 only), a backward product whose reduction axis (the layer's out) is at least
    this long also prunes its own output along the features in its epilogue (mvue_sparse_backward_gemm_pruned), with
    the seed the layer below would have used, so that layer's prune along the features is not launched.  Same bits.
    Returns the list of dW (fp32), top layer first."""
    g = g_top
    grads = []
    ready = None                                          # (values, meta) of the current g along the features, if already made
    fuse_joint = binding.MVUE_JOINT_TABLE if joint is None else joint

    def backward(i, L, values_b, meta_b):
        nonlocal ready
        below = layers[i + 1] if i + 1 < len(layers) else None
        if (prune_in_epilogue_min_k is not None and (n, m) == (2, 4) and L["W"].shape[0] >= prune_in_epilogue_min_k
                and below is not None and below.get("act_grad") is not None and L["W"].shape[1] % 128 == 0
                and fuse_joint in (binding.MVUE_JOINT_TABLE, binding.MVUE_JOINT_SYSTEMATIC)):
            g_next, nv, nm = binding.mvue_sparse_backward_gemm_pruned(values_b, meta_b, L["W"], L["act_grad"],
                                                                      layer_seeds(base_seed, i + 1)[1], next_joint=fuse_joint,
                                                                      next_options=options)
            ready = (nv, nm)
            return g_next
        ready = None
        return binding.mvue_sparse_backward_gemm(values_b, meta_b, L["W"], act_grad=L["act_grad"], out_dtype=torch.bfloat16)

    def prune_features(g, s_bwd):
        if ready is not None:
            return ready
        return binding.mvue_prune(g, n, m, 1, s_bwd, layout=TC, joint=joint, options=options)

    main = torch.cuda.current_stream()
    side = torch.cuda.Stream(priority=-1) if overlap else None
    for i, L in enumerate(layers):
        s_upd, s_bwd = layer_seeds(base_seed, i)
        values, meta = binding.mvue_prune(g, n, m, 0, s_upd, layout=TC, joint=joint, options=options)
        propagate = L.get("act_grad") is not None
        if overlap and propagate:
            dW = torch.empty((values.shape[0], L["h"].shape[1]), dtype=torch.float32, device=g.device)
            ws_bytes = binding.mvue_gemm_workspace_bytes(0, dW.shape[0], dW.shape[1], g.shape[0])
            ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=g.device)
            side.wait_stream(main)
            with torch.cuda.stream(side):
                binding.mvue_sparse_update_gemm(values, meta, L["h"], out=dW, workspace=ws)
            values_b, meta_b = prune_features(g, s_bwd)
            main.wait_stream(side)                       # (values, meta, ws stay referenced until here)
            grads.append(dW)
            g = backward(i, L, values_b, meta_b)
            continue
        grads.append(binding.mvue_sparse_update_gemm(values, meta, L["h"]))
        if propagate:
            values, meta = prune_features(g, s_bwd)
            g = backward(i, L, values, meta)
    return grads

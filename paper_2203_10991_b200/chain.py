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


def backward_update(g_top: torch.Tensor, layers, n: int = 2, m: int = 4, base_seed: int = 0, joint: int | None = None):
    """layers: list (top layer first) of dicts {"W": [out x in] bf16, "h": [T x in] bf16,
    "act_grad": [T x in] bf16 or None (None for the bottom layer: no gradient is propagated further)}.
    joint: the 2:4 law over pairs handed to mvue_prune_joint (None: mvue_prune, the App. A.2 table).
    Returns the list of dW (fp32), top layer first."""
    g = g_top
    grads = []
    for i, L in enumerate(layers):
        s_upd, s_bwd = layer_seeds(base_seed, i)
        values, meta = binding.mvue_prune(g, n, m, 0, s_upd, layout=TC, joint=joint)
        grads.append(binding.mvue_sparse_update_gemm(values, meta, L["h"]))
        if L.get("act_grad") is not None:
            values, meta = binding.mvue_prune(g, n, m, 1, s_bwd, layout=TC, joint=joint)
            g = binding.mvue_sparse_backward_gemm(values, meta, L["W"], act_grad=L["act_grad"],
                                                  out_dtype=torch.bfloat16)
    return grads

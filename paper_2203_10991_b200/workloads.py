"""Seeded synthetic inputs for tests and benchmarks.

Holds no arithmetic of the pruning method: only random tensors with the shapes
and value distributions of the workloads (ReLU-sparse normal, ReLU-sparse
lognormal and Student-t neural gradients; normal activations and weights),
drawn on the host with numpy's PCG64 so that every consumer sees identical
bits.  bf16 tensors are returned as uint16 bit patterns (cast by torch).
"""
from __future__ import annotations

import numpy as np
import torch


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def _chunks(rows: int, cols: int, max_elems: int = 1 << 24):
    step = max(1, max_elems // max(1, cols))
    for r0 in range(0, rows, step):
        yield r0, min(rows, r0 + step)


def gradient(shape, dist: str, seed: int, dtype: str = "bf16") -> np.ndarray:
    """A neural-gradient stand-in g[rows, cols].

    dist: "relu_normal"    N(0,1), each entry zeroed with probability 1/2
          "relu_lognormal" sign * exp(N(0, 2)), each entry zeroed with probability 1/2
          "student_t"      1e-3 * Student-t(nu = 3)
    dtype "f32" returns float32, "bf16" returns uint16 bit patterns.
    Large tensors are drawn in row chunks from one generator, so the result
    depends only on (shape, dist, seed).
    """
    rows, cols = shape
    rng = _rng(seed)
    out = np.empty((rows, cols), dtype=np.float32 if dtype == "f32" else np.uint16)
    for r0, r1 in _chunks(rows, cols):
        n = (r1 - r0, cols)
        if dist == "relu_normal":
            x = rng.standard_normal(n, dtype=np.float32)
            x = np.where(rng.random(n, dtype=np.float32) < 0.5, x, np.float32(0))
        elif dist == "relu_lognormal":
            x = np.exp(2.0 * rng.standard_normal(n, dtype=np.float32))
            x *= np.where(rng.random(n, dtype=np.float32) < 0.5, np.float32(1), np.float32(-1))
            x = np.where(rng.random(n, dtype=np.float32) < 0.5, x, np.float32(0))
        elif dist == "student_t":
            x = (1e-3 * rng.standard_t(3.0, n)).astype(np.float32)
        else:
            raise KeyError(dist)
        x = x.astype(np.float32)
        out[r0:r1] = x if dtype == "f32" else to_bf16_bits(x)
    return out


def normal_bf16(shape, seed: int, std: float = 1.0) -> np.ndarray:
    """Activations / weights / activation derivatives: N(0, std^2) as bf16 bits."""
    rows, cols = shape
    rng = _rng(seed)
    out = np.empty((rows, cols), dtype=np.uint16)
    for r0, r1 in _chunks(rows, cols):
        x = rng.standard_normal((r1 - r0, cols), dtype=np.float32)
        if std != 1.0:
            x *= np.float32(std)
        out[r0:r1] = to_bf16_bits(x)
    return out


# The five workload configurations (shapes only; tensors are drawn on demand).
CONFIGS = {
    "linear_small": dict(T=512, out=256, inp=256, g_dist="relu_normal", g_dtype="f32", seed=0,
                         modes=((1, 2),)),
    "conv_im2col": dict(T=64 * 56 * 56, out=256, inp=2304, g_dist="relu_lognormal", g_dtype="bf16",
                        seed=1, modes=((2, 4), (1, 2))),
    "ffn_768": dict(T=8192, out=3072, inp=768, g_dist="student_t", g_dtype="bf16", seed=2,
                    modes=((2, 4),)),
    "ffn_large": dict(T=16384, out=14336, inp=4096, g_dist="student_t", g_dtype="bf16", seed=3,
                      modes=((2, 4), (1, 2))),
    "mlp_stack": dict(T=32768, out=4096, inp=1024, g_dist="student_t", g_dtype="bf16", seed=4,
                      modes=((2, 4),), layers=12),
}

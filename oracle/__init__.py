"""CPU oracle for MVUE N:M gradient pruning and the products that consume it.

TEST INFRASTRUCTURE ONLY: a plain, slow statement of what the method computes,
written from the paper.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library never does, and the
two share no code.

`mvue_oracle.c` holds the arithmetic (binary32, fixed order, no fused
multiply-add); this module compiles it with gcc on first use and exposes it
through ctypes with numpy arrays.  `theory.py` holds the binary64 closed forms
of the paper (probabilities, marginals, variances) that pin the sampler.
`philox_py.py` is an independent big-integer restatement of the generator.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "mvue_oracle.c"
_LIB = _HERE / "_build" / "libmvue_oracle.so"

_CFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c11", "-fPIC", "-shared", "-fopenmp"]


def build(force: bool = False) -> Path:
    """Compile the C oracle (gcc, no fast-math, no FMA contraction)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        _LIB.parent.mkdir(exist_ok=True)
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(["gcc", *_CFLAGS, str(_SRC), "-o", str(tmp), "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(str(build()))
        u32p = ctypes.POINTER(ctypes.c_uint32)
        L.oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.oracle_philox4x32_10.restype = None
        L.oracle_block_word.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        L.oracle_block_word.restype = ctypes.c_uint32
        L.oracle_uniform24.argtypes = [ctypes.c_uint32]
        L.oracle_uniform24.restype = ctypes.c_float
        L.oracle_bf16_rne.argtypes = [ctypes.c_float]
        L.oracle_bf16_rne.restype = ctypes.c_uint16
        L.oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
        L.oracle_bf16_to_f32.restype = ctypes.c_float
        L.oracle_mvue_1of2.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_uint32,
                                       ctypes.POINTER(ctypes.c_float)]
        L.oracle_mvue_1of2.restype = ctypes.c_int
        L.oracle_mvue_2of4.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_uint32,
                                       ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_float)]
        L.oracle_mvue_2of4.restype = None
        L.oracle_mvue_2of4_systematic.argtypes = L.oracle_mvue_2of4.argtypes
        L.oracle_mvue_2of4_cases.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_uint32,
                                             ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_double)]
        L.oracle_mvue_2of4_cases.restype = ctypes.c_int
        L.oracle_sweep_2of4_cases.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.POINTER(ctypes.c_uint64),
                                              ctypes.POINTER(ctypes.c_double)]
        L.oracle_sweep_2of4_cases.restype = ctypes.c_int
        L.oracle_mvue_2of4_systematic.restype = None
        L.oracle_mvue_2of4_approx.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_uint32, ctypes.c_uint32,
                                              ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_float)]
        L.oracle_mvue_2of4_approx.restype = None
        L.oracle_block_word_pair.argtypes = [ctypes.c_uint64, ctypes.c_uint64, u32p]
        L.oracle_block_word_pair.restype = None
        L.oracle_sweep_approx24.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_uint64),
                                            ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_float)]
        L.oracle_sweep_approx24.restype = None
        L.oracle_mvue_1of4.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_uint32, ctypes.POINTER(ctypes.c_float)]
        L.oracle_mvue_1of4.restype = ctypes.c_int
        L.oracle_sweep_1of4.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_uint64),
                                        ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
        L.oracle_sweep_1of4.restype = None
        L.oracle_prune.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
                                   ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                   ctypes.c_uint64, ctypes.c_int64, ctypes.c_int64,
                                   ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
        L.oracle_prune.restype = ctypes.c_int
        L.oracle_prune_rounded.argtypes = L.oracle_prune.argtypes + [ctypes.c_int]
        L.oracle_prune_rounded.restype = ctypes.c_int
        L.oracle_prune_opts.argtypes = L.oracle_prune.argtypes + [ctypes.c_int, ctypes.c_int]
        L.oracle_prune_opts.restype = ctypes.c_int
        L.oracle_block_word16.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        L.oracle_block_word16.restype = ctypes.c_uint32
        L.oracle_block_word_pair16.argtypes = [ctypes.c_uint64, ctypes.c_uint64, u32p]
        L.oracle_block_word_pair16.restype = None
        L.oracle_bf16_sr.argtypes = [ctypes.c_float, ctypes.c_uint16]
        L.oracle_bf16_sr.restype = ctypes.c_uint16
        L.oracle_rounding_bits.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int]
        L.oracle_rounding_bits.restype = ctypes.c_uint16
        L.oracle_approx_4of8.argtypes = [ctypes.POINTER(ctypes.c_float), u32p, ctypes.POINTER(ctypes.c_int),
                                         ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float)]
        L.oracle_approx_4of8.restype = None
        L.oracle_approx_4of8_ordered.argtypes = L.oracle_approx_4of8.argtypes + [ctypes.POINTER(ctypes.c_int)]
        L.oracle_approx_4of8_ordered.restype = None
        L.oracle_block_words4.argtypes = [ctypes.c_uint64, ctypes.c_uint64, u32p]
        L.oracle_block_words4.restype = None
        L.oracle_prune_4of8.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                        ctypes.c_int, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int64,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        L.oracle_prune_4of8.restype = ctypes.c_int
        L.oracle_unpack.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                    ctypes.c_void_p]
        L.oracle_unpack.restype = None
        L.oracle_gemm.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                  ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64,
                                  ctypes.c_void_p, ctypes.c_int]
        L.oracle_gemm.restype = None
        L.oracle_gemm_entry.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                        ctypes.c_int64, ctypes.c_int64]
        L.oracle_gemm_entry.restype = ctypes.c_double
        L.oracle_sweep_2of4.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.POINTER(ctypes.c_uint64),
                                        ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
        L.oracle_sweep_2of4.restype = None
        L.oracle_sweep_1of2.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.POINTER(ctypes.c_uint64),
                                        ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
        L.oracle_sweep_1of2.restype = None
        _lib = L
    return _lib


def host_threads() -> int:
    return len(os.sched_getaffinity(0))


# --------------------------------------------------------------------------
# thin numpy wrappers
# --------------------------------------------------------------------------
def philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (ctypes.c_uint32 * 4)()
    lib().oracle_philox4x32_10(c, k, o)
    return tuple(int(x) for x in o)


def block_word(seed: int, q: int) -> int:
    return int(lib().oracle_block_word(seed & (2**64 - 1), q))


def block_word16(seed: int, q: int) -> int:
    """The word of block q when blocks draw sixteen bits each: those bits in the top half, zero below."""
    return int(lib().oracle_block_word16(seed & (2**64 - 1), q))


def block_word_pair16(seed: int, q: int):
    out = (ctypes.c_uint32 * 2)()
    lib().oracle_block_word_pair16(seed & (2**64 - 1), q, out)
    return int(out[0]), int(out[1])


def uniform24(word: int) -> float:
    return float(lib().oracle_uniform24(word & 0xFFFFFFFF))


def bf16_rne(x: np.ndarray) -> np.ndarray:
    """binary32 array -> bf16 bit patterns (uint16), element by element."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    f = lib().oracle_bf16_rne
    return np.fromiter((f(float(v)) for v in x.ravel()), dtype=np.uint16, count=x.size).reshape(x.shape)


def bf16_to_f32(h: np.ndarray) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.uint16)
    return (h.astype(np.uint32) << 16).view(np.float32)


def mvue_1of2(a1: float, a2: float, word: int):
    kept = ctypes.c_float()
    idx = lib().oracle_mvue_1of2(a1, a2, word & 0xFFFFFFFF, ctypes.byref(kept))
    return int(idx), float(kept.value)


JOINT_TABLE, JOINT_SYSTEMATIC = 0, 1      # 2:4 law over pairs: App. A.2 table / systematic sampling
JOINT_APPROX = 2                          # approx-MVUE 2:4 of Sec. 4.4 (two sequential draws, two words per block)


def mvue_2of4(a, word: int, joint: int = JOINT_TABLE):
    arr = (ctypes.c_float * 4)(*[float(x) for x in a])
    idx = (ctypes.c_int * 2)()
    val = (ctypes.c_float * 2)()
    fn = lib().oracle_mvue_2of4 if joint == JOINT_TABLE else lib().oracle_mvue_2of4_systematic
    fn(arr, word & 0xFFFFFFFF, idx, val)
    return (int(idx[0]), int(idx[1])), (float(val[0]), float(val[1]))


def mvue_2of4_cases(a, word: int):
    """App. A.2 case by case in binary64: (case number, (idx0, idx1), (val0, val1)); case -1 (nothing else
    computed) for a block with fewer than two non-zeros, which the appendix does not cover."""
    arr = (ctypes.c_float * 4)(*[float(x) for x in a])
    idx = (ctypes.c_int * 2)()
    val = (ctypes.c_double * 2)()
    which = lib().oracle_mvue_2of4_cases(arr, word & 0xFFFFFFFF, idx, val)
    if which < 0:
        return -1, None, None
    return int(which), (int(idx[0]), int(idx[1])), (float(val[0]), float(val[1]))


def sweep_2of4_cases(a, mistake: int = 0):
    """All 2^24 eps through the case-by-case statement of App. A.2 and through mvue_2of4:
    (case number, draws on which the kept pairs differ, largest relative difference of the kept values).
    mistake = 1, 2, 3 plants an error in that case's formulas of the case-by-case statement (power check)."""
    arr = (ctypes.c_float * 4)(*[float(x) for x in a])
    diff = ctypes.c_uint64()
    rel = ctypes.c_double()
    which = lib().oracle_sweep_2of4_cases(arr, int(mistake), ctypes.byref(diff), ctypes.byref(rel))
    return int(which), int(diff.value), float(rel.value)


def mvue_2of4_approx(a, word1: int, word2: int):
    """Sec. 4.4 on one block: ((idx0, idx1), (val0, val1)) with idx0 < idx1."""
    arr = (ctypes.c_float * 4)(*[float(x) for x in a])
    idx = (ctypes.c_int * 2)()
    val = (ctypes.c_float * 2)()
    lib().oracle_mvue_2of4_approx(arr, word1 & 0xFFFFFFFF, word2 & 0xFFFFFFFF, idx, val)
    return (int(idx[0]), int(idx[1])), (float(val[0]), float(val[1]))


def block_word_pair(seed: int, q: int):
    out = (ctypes.c_uint32 * 2)()
    lib().oracle_block_word_pair(seed & (2**64 - 1), q, out)
    return int(out[0]), int(out[1])


def mvue_1of4(a, word: int):
    """MVUE 1:4 on one block: (surviving position, its new value)."""
    arr = (ctypes.c_float * 4)(*[float(x) for x in a])
    kept = ctypes.c_float()
    i = lib().oracle_mvue_1of4(arr, word & 0xFFFFFFFF, ctypes.byref(kept))
    return int(i), float(kept.value)


def sweep_1of4(a):
    """Frequencies of the four outcomes, mean of theta(a) and block variance over all 2^24 eps."""
    arr = (ctypes.c_float * 4)(*[float(x) for x in a])
    counts = (ctypes.c_uint64 * 4)()
    sums = (ctypes.c_double * 4)()
    sq = ctypes.c_double()
    lib().oracle_sweep_1of4(arr, counts, sums, ctypes.byref(sq))
    n = float(1 << 24)
    return (np.array(list(counts), dtype=np.float64) / n, np.array(list(sums)) / n, sq.value / n)


def packed_shapes(rows: int, cols: int, axis: int):
    mrows, k = (rows, cols) if axis == 1 else (cols, rows)
    return (mrows, k // 2), (mrows, k // 8)


def bf16_sr(x: float, r: int) -> int:
    """Stochastic rounding of a binary32 value to bf16 bits with the 16 random bits r."""
    return int(lib().oracle_bf16_sr(float(x), r & 0xFFFF))


def rounding_bits(seed: int, unit: int, slot: int) -> int:
    return int(lib().oracle_rounding_bits(seed & (2**64 - 1), unit, slot))


def prune(g: np.ndarray, n: int, m: int, axis: int, seed: int, *, k_total: int | None = None,
          k_offset: int = 0, threads: int = 1, joint: int = JOINT_TABLE, stochastic_rounding: bool = False,
          eps16: bool = False):
    """MVUE n:m prune + pack of a 2-D array (float32, or uint16 holding bf16 bits).
    joint: the 2:4 estimator (JOINT_TABLE: App. A.2; JOINT_SYSTEMATIC; JOINT_APPROX: Sec. 4.4); ignored for 1:2.
    stochastic_rounding: survivors are rounded to bf16 stochastically (unbiased storage) instead of to nearest.
    eps16: sixteen random bits per block (one generator call per eight blocks) instead of thirty-two.

    Returns (values uint16 [Mrows, K/2], meta uint8 [Mrows, K/8]) in canonical form.
    """
    assert g.ndim == 2 and g.dtype in (np.float32, np.uint16)
    g = np.ascontiguousarray(g)
    rows, cols = g.shape
    vshape, mshape = packed_shapes(rows, cols, axis)
    k = cols if axis == 1 else rows
    values = np.zeros(vshape, dtype=np.uint16)
    meta = np.zeros(mshape, dtype=np.uint8)
    rc = lib().oracle_prune_opts(g.ctypes.data, int(g.dtype == np.uint16), rows, cols, cols, n, m, axis,
                                 seed & (2**64 - 1), k if k_total is None else k_total, k_offset,
                                 values.ctypes.data, meta.ctypes.data, max(1, threads), int(joint),
                                 int(bool(stochastic_rounding)), int(bool(eps16)))
    if rc != 0:
        raise ValueError("oracle_prune: unsupported N:M or shape")
    return values, meta


def unpack(values: np.ndarray, meta: np.ndarray) -> np.ndarray:
    """Canonical packed operand -> dense float32 A[Mrows, K]."""
    values = np.ascontiguousarray(values, dtype=np.uint16)
    meta = np.ascontiguousarray(meta, dtype=np.uint8)
    mrows, kh = values.shape
    dense = np.empty((mrows, 2 * kh), dtype=np.float32)
    lib().oracle_unpack(values.ctypes.data, meta.ctypes.data, mrows, 2 * kh, dense.ctypes.data)
    return dense


def gemm(A: np.ndarray, B: np.ndarray, E: np.ndarray | None = None, threads: int = 1) -> np.ndarray:
    """C = A @ B (* E), A float32 [M,K], B / E uint16 bf16 bits [K,N] / [M,N]; float64 result."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    B = np.ascontiguousarray(B, dtype=np.uint16)
    M, K = A.shape
    assert B.shape[0] == K
    N = B.shape[1]
    C = np.empty((M, N), dtype=np.float64)
    if E is not None:
        E = np.ascontiguousarray(E, dtype=np.uint16)
        assert E.shape == (M, N)
    lib().oracle_gemm(A.ctypes.data, M, K, B.ctypes.data, N, N,
                      None if E is None else E.ctypes.data, N, C.ctypes.data, max(1, threads))
    return C


def gemm_entry(A_row: np.ndarray, B: np.ndarray, j: int) -> float:
    A_row = np.ascontiguousarray(A_row, dtype=np.float32)
    B = np.ascontiguousarray(B, dtype=np.uint16)
    return float(lib().oracle_gemm_entry(A_row.ctypes.data, A_row.size, B.ctypes.data, B.shape[1], j))


PAIRS = ((0, 1), (0, 2), (0, 3), (1, 2), (1, 3), (2, 3))


def sweep_2of4(a, joint: int = JOINT_TABLE):
    """Frequencies of the six outcomes, mean of theta(a) and block variance over all 2^24 eps."""
    arr = (ctypes.c_float * 4)(*[float(x) for x in a])
    counts = (ctypes.c_uint64 * 6)()
    sums = (ctypes.c_double * 4)()
    sq = ctypes.c_double()
    lib().oracle_sweep_2of4(arr, int(joint), counts, sums, ctypes.byref(sq))
    n = float(1 << 24)
    return (np.array([c for c in counts], dtype=np.float64) / n,
            np.array([s for s in sums]) / n, sq.value / n)


def sweep_1of2(a1: float, a2: float):
    counts = (ctypes.c_uint64 * 2)()
    sums = (ctypes.c_double * 2)()
    sq = ctypes.c_double()
    lib().oracle_sweep_1of2(a1, a2, counts, sums, ctypes.byref(sq))
    n = float(1 << 24)
    return (np.array([c for c in counts], dtype=np.float64) / n,
            np.array([s for s in sums]) / n, sq.value / n)


def sweep_approx24(a):
    """Sec. 4.4 sampler, one draw at a time over all 2^24 values of each uniform:
    (P[first = i], P[second = j | first = i] (rows of never-drawn i are NaN), value of k when it survives)."""
    arr = (ctypes.c_float * 4)(*[float(x) for x in a])
    first = (ctypes.c_uint64 * 4)()
    second = (ctypes.c_uint64 * 16)()
    val = (ctypes.c_float * 4)()
    lib().oracle_sweep_approx24(arr, first, second, val)
    n = float(1 << 24)
    f = np.array(list(first), dtype=np.float64) / n
    sec = np.array(list(second), dtype=np.float64).reshape(4, 4) / n
    sec[f == 0] = np.nan
    return f, sec, np.array(list(val), dtype=np.float64)


# ------------------------------------------------------------------ approx-4:8 (prune only) -------
def approx_4of8(a, words):
    """Approx-4:8 on one block of eight: (positions ascending, new values, the eight inclusion probabilities)."""
    arr = (ctypes.c_float * 8)(*[float(x) for x in a])
    w = (ctypes.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in words])
    idx = (ctypes.c_int * 4)()
    val = (ctypes.c_float * 4)()
    p = (ctypes.c_float * 8)()
    lib().oracle_approx_4of8(arr, w, idx, val, p)
    return tuple(int(i) for i in idx), tuple(float(v) for v in val), np.array(list(p), dtype=np.float64)


def approx_4of8_order(a, words):
    """The four positions of approx-4:8 in the order they were drawn."""
    arr = (ctypes.c_float * 8)(*[float(x) for x in a])
    w = (ctypes.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in words])
    idx = (ctypes.c_int * 4)()
    val = (ctypes.c_float * 4)()
    p = (ctypes.c_float * 8)()
    order = (ctypes.c_int * 4)()
    lib().oracle_approx_4of8_ordered(arr, w, idx, val, p, order)
    return tuple(int(i) for i in order)


def block_words4(seed: int, q: int):
    out = (ctypes.c_uint32 * 4)()
    lib().oracle_block_words4(seed & (2**64 - 1), q, out)
    return tuple(int(x) for x in out)


def prune_4of8(g: np.ndarray, axis: int, seed: int, *, k_total: int | None = None, k_offset: int = 0, threads: int = 1):
    """Approx-4:8 prune of a 2-D array: (values uint16 [Mrows, K/2], mask uint8 [Mrows, K/8], bit k = element k kept)."""
    assert g.ndim == 2 and g.dtype in (np.float32, np.uint16)
    g = np.ascontiguousarray(g)
    rows, cols = g.shape
    mrows, k = (rows, cols) if axis == 1 else (cols, rows)
    values = np.zeros((mrows, k // 2), dtype=np.uint16)
    mask = np.zeros((mrows, k // 8), dtype=np.uint8)
    rc = lib().oracle_prune_4of8(g.ctypes.data, int(g.dtype == np.uint16), rows, cols, cols, axis, seed & (2**64 - 1),
                                 k if k_total is None else k_total, k_offset, values.ctypes.data, mask.ctypes.data,
                                 max(1, threads))
    if rc != 0:
        raise ValueError("oracle_prune_4of8: unsupported shape")
    return values, mask


def unpack_4of8(values: np.ndarray, mask: np.ndarray) -> np.ndarray:
    """Dense float32 A[Mrows, K] from the approx-4:8 packed form (plain numpy: no arithmetic of the method)."""
    mrows, kh = values.shape
    dense = np.zeros((mrows, 2 * kh), dtype=np.float32)
    vals = bf16_to_f32(values)
    for r in range(mrows):
        for j in range(kh // 4):
            pos = [k for k in range(8) if mask[r, j] >> k & 1]
            for e, k in enumerate(pos):
                dense[r, 8 * j + k] = vals[r, 4 * j + e]
    return dense

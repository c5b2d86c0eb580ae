"""Test-side restatement of the tensor-core metadata order (MVUE_LAYOUT_TC in include/mvue.h),
written from the layout's definition and used to carry the oracle's canonical metadata into the
order the GEMMs consume.  Pure index arithmetic, no method arithmetic."""
import numpy as np


def canonical_to_tc(meta: np.ndarray, pad_pattern: int = 0x44) -> np.ndarray:
    """meta uint8 [Mrows, K/8] (canonical) -> uint8 [ceil(Mrows/128)*128 * K/8] flat, TC order."""
    mrows, kb = meta.shape
    K = kb * 8
    assert K % 128 == 0
    mpad = (mrows + 127) // 128 * 128
    kblocks = K // 128
    out = np.full(mpad * kb, pad_pattern, dtype=np.uint8)
    words = meta.reshape(mrows, K // 16, 2)                       # 16-bit units: (row, strip)
    r = np.arange(mrows)[:, None]
    strip = np.arange(K // 16)[None, :]
    rl, st = r % 128, strip % 8
    lane = (rl % 8) + 8 * (st % 2) + 16 * (rl // 16)
    off = ((r // 128) * kblocks + strip // 8) * 2048 + lane * 16 + (st // 2) * 4 + ((rl // 8) % 2) * 2
    out[off] = words[:, :, 0]
    out[off + 1] = words[:, :, 1]
    return out


def tc_to_canonical(tc: np.ndarray, mrows: int, K: int) -> np.ndarray:
    kb = K // 8
    kblocks = K // 128
    r = np.arange(mrows)[:, None]
    strip = np.arange(K // 16)[None, :]
    rl, st = r % 128, strip % 8
    lane = (rl % 8) + 8 * (st % 2) + 16 * (rl // 16)
    off = ((r // 128) * kblocks + strip // 8) * 2048 + lane * 16 + (st // 2) * 4 + ((rl // 8) % 2) * 2
    flat = tc.reshape(-1)
    words = np.stack([flat[off], flat[off + 1]], axis=2)
    return words.reshape(mrows, kb)

"""Host-side arithmetic for data parallelism over tokens.

The token axis is the reduction axis K of the update product, so each rank prunes and multiplies its
own token shard and the partial dW are summed by one all-reduce.  Shard boundaries are multiples of
128 tokens (the K granularity of the packed operand), and a shard pruned with the global `k_total`
and its own `k_offset` draws exactly the random words the unsharded tensor would.
"""
from __future__ import annotations

GRANULE = 128


def token_shard(total_tokens: int, world_size: int, rank: int) -> tuple[int, int]:
    """(offset, length) of rank's token shard; lengths differ by at most one granule, sum to the total."""
    if total_tokens % GRANULE != 0:
        raise ValueError(f"token count must be a multiple of {GRANULE}")
    if not 0 <= rank < world_size:
        raise ValueError("rank out of range")
    granules = total_tokens // GRANULE
    base, extra = divmod(granules, world_size)
    start = rank * base + min(rank, extra)
    count = base + (1 if rank < extra else 0)
    return start * GRANULE, count * GRANULE

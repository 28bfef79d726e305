"""Multi-GPU partition of one attention layer: by KV head group, with no exchange on the data path.

Every (sequence, KV head) pair is independent through the gate, the mask and the attention (query heads
g*G .. g*G+G-1 read only KV head g), so a rank takes a contiguous range of KV heads, the matching query heads, and runs
the same three library calls on its slice.  Outputs are concatenated along the head axis.  Host logic only.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class HeadShard:
    rank: int
    world: int
    kv_lo: int          # first KV head of this rank
    kv_hi: int          # one past the last
    group: int          # query heads per KV head

    @property
    def q_lo(self) -> int:
        return self.kv_lo * self.group

    @property
    def q_hi(self) -> int:
        return self.kv_hi * self.group

    @property
    def num_kv_heads(self) -> int:
        return self.kv_hi - self.kv_lo

    @property
    def num_q_heads(self) -> int:
        return self.q_hi - self.q_lo


def kv_head_shard(num_q_heads: int, num_kv_heads: int, world: int, rank: int) -> HeadShard:
    """Balanced contiguous ranges: the first (num_kv_heads % world) ranks take one head more.  A rank may be empty
    when world > num_kv_heads."""
    if num_q_heads % num_kv_heads:
        raise ValueError("num_q_heads must be a multiple of num_kv_heads")
    if not 0 <= rank < world:
        raise ValueError("rank out of range")
    base, extra = divmod(num_kv_heads, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return HeadShard(rank, world, lo, hi, num_q_heads // num_kv_heads)


def slice_inputs(shard: HeadShard, q, k, v, wq, wk):
    """Views of [T, H, d] tensors / [H, d, dg] weights restricted to the rank's heads (numpy or torch)."""
    return (q[:, shard.q_lo:shard.q_hi], k[:, shard.kv_lo:shard.kv_hi], v[:, shard.kv_lo:shard.kv_hi],
            wq[shard.q_lo:shard.q_hi], wk[shard.kv_lo:shard.kv_hi])


def concat_heads(parts, axis: int = 1):
    """Inverse of the head split for outputs laid out [T, Hq_local, d] (axis 1) or [Hq_local, T] (axis 0)."""
    return np.concatenate([p for p in parts if p.shape[axis] > 0], axis=axis)

"""One layer's state sharded by KV head over the ranks of a torch.distributed job.

Orchestration only: every step of the path runs in the CUDA library.  Each
rank holds n_kv_heads / world KV heads and the query heads that read them;
the only exchange per token is the sum over ranks of one fp32 vector of
capacity+1 entries per sequence (Algorithm 1's mean over heads is a sum), done
here with an all-reduce on the caller's stream between the library's two calls
tova_decode_step_scores and tova_decode_step_commit.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist

from .binding import TOVA_DTYPE_BF16, TovaCache


class ShardedTovaLayer:
    """This rank's share of one layer.  q, k, v passed to step() are the rank's
    own heads: q [B, H/world, D], k and v [B, Hkv/world, D]."""

    def __init__(self, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int, capacity: int,
                 dtype: int = TOVA_DTYPE_BF16, device: str = "cuda:0", rank: Optional[int] = None,
                 world: Optional[int] = None, group=None):
        self.group = group
        self.rank = dist.get_rank(group) if rank is None else rank
        self.world = dist.get_world_size(group) if world is None else world
        if n_kv_heads % self.world:
            raise ValueError("the KV heads must divide evenly over the ranks")
        self.cache = TovaCache(batch, n_q_heads // self.world, n_kv_heads // self.world, head_dim, capacity,
                               dtype=dtype, device=device)
        ld = (capacity + 1 + 3) // 4 * 4
        self.table = torch.zeros(batch, ld, dtype=torch.float32, device=device)
        tables = [self.table if r == self.rank else None for r in range(self.world)]
        self.cache.tova_cache_set_shard(self.rank, self.world, n_q_heads, tables, None)
        self.capacity = capacity

    def step(self, q, k, v, pos: int, out, evicted_pos=None) -> None:
        full = self.cache.tova_cache_len() == self.capacity
        self.cache.tova_decode_step_scores(q, k, v, pos, out)
        if full and self.world > 1:                 # the one exchange of the step
            dist.all_reduce(self.table, op=dist.ReduceOp.SUM, group=self.group)
        self.cache.tova_decode_step_commit(k, v, evicted_pos)

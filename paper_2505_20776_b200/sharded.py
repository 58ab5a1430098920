"""KV-head sharding of one sequence over several GPUs (one process per GPU).

Verification attention is independent per KV head: a rank that holds Hkv/N KV heads with their G query
heads each computes O, lse and its heads' chunk masses locally with the ordinary library calls.  The
only exchange of the whole path is the head-mean of the chunk scores that retrieval ranks: one
all-reduce of the fp32 block [T][ceil(L/C)] (123 KB at a 16K prefix), over NCCL on GPUs (gloo in the CPU
tests).  Every rank gets the same reduced block, so the (deterministic) selection gives the same chunk
indices everywhere and each rank gathers its own heads of the draft cache; no other collective is needed.

Marshalling and the collective only: all arithmetic of the path stays in the library's kernels.
"""
from __future__ import annotations

from typing import Dict, Optional

import torch
import torch.distributed as dist

from .hotpath import HotPath


def head_shard(n_q_heads: int, n_kv_heads: int, rank: int, world: int):
    """Slices (query heads, KV heads) of this rank: consecutive KV heads with their query heads."""
    if n_kv_heads % world != 0:
        raise ValueError("the number of KV heads must be a multiple of the number of ranks")
    g = n_q_heads // n_kv_heads
    kv = n_kv_heads // world
    return slice(rank * kv * g, (rank + 1) * kv * g), slice(rank * kv, (rank + 1) * kv)


def combine_scores(local_score: torch.Tensor, group=None) -> torch.Tensor:
    """In place: local head-mean chunk scores of equal-sized head shards -> head-mean over all heads.

    local_score is (1/Hq_local) * sum over this rank's heads; with N equal shards the mean over all heads
    is the mean of the ranks' blocks: an all-reduce (sum) and one scaling by 1/N.
    """
    world = dist.get_world_size(group)
    if world > 1:
        dist.all_reduce(local_score, op=dist.ReduceOp.SUM, group=group)
        local_score.mul_(1.0 / world)
    return local_score


class ShardedHotPath:
    """The calls of Algorithm 1's retrieval step for the KV-head shard of this rank."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, n_tree: int, chunk_size: int, top_k: int,
                 max_prefix: int, draft_kv_heads: int, draft_head_dim: Optional[int] = None, draft_layers: int = 1,
                 device="cuda:0", group=None):
        self.group = group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.q_heads, self.kv_heads = head_shard(n_q_heads, n_kv_heads, self.rank, self.world)
        if draft_kv_heads % self.world != 0:
            raise ValueError("the draft model's KV heads must be a multiple of the number of ranks")
        self.local = HotPath(n_q_heads // self.world, n_kv_heads // self.world, head_dim, n_tree, chunk_size, top_k,
                             max_prefix, draft_layers=draft_layers, draft_kv_heads=draft_kv_heads // self.world,
                             draft_head_dim=draft_head_dim, device=device)

    def verify_attn(self, t_local: Dict[str, torch.Tensor], parent: torch.Tensor, prefix_len: int,
                    want_score: bool) -> None:
        """t_local holds this rank's heads only (Q [T][Hq/N][D], K/V [.][Hkv/N][D])."""
        self.local.verify_attn(t_local, parent, prefix_len, want_score)
        if want_score:
            combine_scores(self.local.chunk_score(prefix_len), self.group)

    def select_gather(self, row: int, prefix_len: int, draft_K_local: torch.Tensor, draft_V_local: torch.Tensor) -> None:
        """Same indices on every rank (the reduced scores are identical); each rank copies its draft heads."""
        self.local.select_gather(row, prefix_len, draft_K_local, draft_V_local)

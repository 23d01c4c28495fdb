"""sd_verify over logits that are split along the vocabulary across the ranks of a process
group (a tensor-parallel LM head): four library calls per rank with two small all-gathers
and one max-reduce between them.  Plumbing only: every number is produced by the kernels.

Rank g holds columns ``[v0, v0 + Vs)`` of every p and q row; `vocab_shards` gives the split
this module assumes when none is passed (equal parts, boundaries on 16-byte multiples).
"""
from __future__ import annotations

from typing import List, Tuple

import torch

from . import binding as _b


def vocab_shards(V: int, G: int, elem_bytes: int = 2) -> List[Tuple[int, int]]:
    """(v0, Vs) of every rank: contiguous, in rank order, covering [0, V); interior
    boundaries fall on multiples of 16 bytes so that every shard row can start aligned."""
    if V <= 0 or G <= 0:
        raise ValueError("V and G must be positive")
    vec = 16 // elem_bytes
    units = (V + vec - 1) // vec
    if units < G:
        raise ValueError(f"a vocabulary of {V} cannot be cut into {G} non-empty aligned shards")
    bounds = [min(V, (units * g // G) * vec) for g in range(G)] + [V]
    return [(bounds[g], bounds[g + 1] - bounds[g]) for g in range(G)]


class DistExchange:
    """The collectives of the sharded path on a torch.distributed process group (NCCL for CUDA
    tensors, gloo for host tensors)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist = dist
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        """[...] on every rank -> [G, ...] in rank order."""
        flat = t.contiguous().view(-1)
        out = torch.empty((self.world * flat.numel(),), dtype=t.dtype, device=t.device)
        self._dist.all_gather_into_tensor(out, flat, group=self.group)
        return out.view((self.world,) + tuple(t.shape))

    def all_reduce_max(self, t: torch.Tensor) -> torch.Tensor:
        self._dist.all_reduce(t, op=self._dist.ReduceOp.MAX, group=self.group)
        return t


def sd_verify_sharded(p_shard, q_shard, V: int, v0: int, draft_tokens, uniforms, ws: _b.Workspace,
                      exchange, extras: bool = True, fused: bool = True):
    """p_shard [B,Kp,Vs], q_shard [B,K,Vs] (rows may be strided), draft_tokens i32 [B,K] with
    whole-vocabulary ids, uniforms f32 [B,K+1]; `exchange` has rank, world, all_gather and
    all_reduce_max (a `DistExchange`).  Returns what `sd_verify` returns for the whole rows,
    the same on every rank.  `ws` must hold workspace_bytes(OP_SD_SHARD, B, K, Vs)."""
    B, Kp, Vs = p_shard.shape
    dt = _b._dt(p_shard)
    stats = _b.sd_shard_stats(p_shard, q_shard, v0, draft_tokens, ws)
    all_stats = exchange.all_gather(stats)
    if fused:     # decision and shard weights in one launch
        out, weights = _b.sd_shard_decide_weights(p_shard, q_shard, all_stats, draft_tokens, uniforms, V, ws,
                                                  extras=extras)
    else:
        out = _b.sd_shard_decide(all_stats, draft_tokens, uniforms, V, Vs, Kp, dt, ws, extras=extras)
        weights = _b.sd_shard_weights(p_shard, q_shard, out["accepted_len"], uniforms, ws)
    all_weights = exchange.all_gather(weights)
    out.update(_b.sd_shard_draw(p_shard, q_shard, v0, all_weights, all_stats, exchange.rank,
                                out["accepted_len"], uniforms, ws, extras=extras))
    exchange.all_reduce_max(out["correction_token"])
    return out

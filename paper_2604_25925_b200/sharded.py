"""Vocabulary-sharded verify step: the four local phases of the C ABI (``sgbv_shard_*``) with the three exchanges
between them.

Every rank holds the logits of a contiguous vocabulary range (ascending with the rank).  The exchanges are an
all-gather of the row statistics, an all-gather of the row sums and a max-all-reduce of the token matrix: a few KB
each.  ``verify`` runs one rank's side over ``torch.distributed`` (NCCL on GPUs); ``verify_all_ranks_on_one_device``
runs every rank's side in lockstep on one device, the exchanges being a stack and a maximum: no kernel waits for
another rank, so this is the same computation and is how the single-GPU tests check it.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch

from . import binding


class TorchExchange:
    """The three collectives over a ``torch.distributed`` process group."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist = dist
        self.group = group
        self.world_size = dist.get_world_size(group)
        self.rank = dist.get_rank(group)

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        out = torch.empty((self.world_size * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        self.dist.all_gather_into_tensor(out, t.contiguous(), group=self.group)   # rank r's part at rows [r*n, (r+1)*n)
        return out.view((self.world_size,) + tuple(t.shape))

    def all_reduce_max(self, t: torch.Tensor) -> torch.Tensor:
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX, group=self.group)
        return t


def shard_bounds(V: int, n_ranks: int, multiple: int = 8) -> List[Tuple[int, int]]:
    """Contiguous vocabulary ranges, near-equal, starts on a multiple of `multiple` entries."""
    per = -(-V // n_ranks)
    per = -(-per // multiple) * multiple
    return [(min(V, r * per), min(V, (r + 1) * per)) for r in range(n_ranks)]


def verify(target_shard, draft_shard, draft_tokens, uniforms, temperature: float, v_begin: int, V: int,
           exchange) -> binding.VerifyOutput:
    """One rank's side of the step.  `exchange` supplies rank, all_gather and all_reduce_max."""
    B, K, g1, Vs = target_shard.shape
    ws = torch.empty(binding.sgbv_shard_workspace_bytes(B, K, g1 - 1, Vs, binding._dtype_code(target_shard)),
                     dtype=torch.uint8, device=target_shard.device)
    stats = binding.sgbv_shard_stats(target_shard, draft_shard, draft_tokens, v_begin, V, temperature)
    stats_all = exchange.all_gather(stats)
    sums = binding.sgbv_shard_sums(target_shard, draft_shard, temperature, stats_all, ws)
    sums_all = exchange.all_gather(sums)
    out = binding.sgbv_shard_decide(draft_tokens, uniforms, Vs, temperature, stats_all, sums_all, ws)
    binding.sgbv_shard_draw(target_shard, draft_shard, v_begin, temperature, exchange.rank, ws, out.tokens)
    exchange.all_reduce_max(out.tokens)
    return out


def verify_all_ranks_on_one_device(shards: Sequence[Tuple[torch.Tensor, torch.Tensor, int]], draft_tokens, uniforms,
                                   temperature: float, V: int) -> List[binding.VerifyOutput]:
    """Every rank's side, phase by phase, on one device.  shards[r] = (target_shard, draft_shard, v_begin)."""
    R = len(shards)
    code = binding._dtype_code(shards[0][0])
    wss = []
    for zq, _, _ in shards:
        B, K, g1, Vs = zq.shape
        wss.append(torch.empty(binding.sgbv_shard_workspace_bytes(B, K, g1 - 1, Vs, code), dtype=torch.uint8,
                               device=zq.device))
    stats_all = torch.stack([binding.sgbv_shard_stats(zq, zp, draft_tokens, vb, V, temperature)
                             for zq, zp, vb in shards]).contiguous()
    sums_all = torch.stack([binding.sgbv_shard_sums(zq, zp, temperature, stats_all, wss[r])
                            for r, (zq, zp, _) in enumerate(shards)]).contiguous()
    outs = [binding.sgbv_shard_decide(draft_tokens, uniforms, shards[r][0].shape[-1], temperature, stats_all, sums_all,
                                      wss[r]) for r in range(R)]
    for r, (zq, zp, vb) in enumerate(shards):
        binding.sgbv_shard_draw(zq, zp, vb, temperature, r, wss[r], outs[r].tokens)
    # the max-all-reduce of the token matrices, through the C ABI's outputs only
    reduced = torch.stack([o.tokens for o in outs]).amax(dim=0)
    for o in outs:
        o.tokens.copy_(reduced)
    return outs

"""The verification round for an edge whose vocabulary is sharded over the ranks of a process group.

Rank g holds entries [v_begin, v_begin + V_shard) of every target logit row (what a tensor-parallel
LM head leaves on each GPU) and the same slice of the device's rows Q_i.  One round is five library
calls per rank with two small all-gathers between them (a few bytes per row: partial sums, then
masses) and a final max over ranks for the token.  The exchanges are plain torch.distributed
collectives on this rank's own tensors; no kernel of the library touches another GPU's memory.

Argument marshalling and collectives only: every step of the method runs in the library's kernels.
"""
from __future__ import annotations

from typing import Dict, Optional

import torch
import torch.distributed as dist


def all_gather_shards(t: torch.Tensor, group=None) -> torch.Tensor:
    """A tensor of the same shape on each of the G ranks -> [G, ...] in rank order, on every rank."""
    world = dist.get_world_size(group)
    parts = [torch.empty_like(t) for _ in range(world)]
    dist.all_gather(parts, t.contiguous(), group=group)
    return torch.stack(parts)


def verify_round_vocab_sharded(logits_shard: torch.Tensor, draft_tokens: torch.Tensor, draft_q_tok: torch.Tensor,
                               uniforms: torch.Tensor, draft_q_shard: Optional[torch.Tensor],
                               uniforms_rs: torch.Tensor, temperature: float, v_begin: int, V: int,
                               group=None) -> Dict[str, torch.Tensor]:
    """One round on this rank's shard.  logits_shard [B, gamma+1, V_shard], draft_q_shard
    [B, gamma, V_shard] (CUDA); the per-sequence inputs are replicated on every rank.  Returns
    accept_len, token (the same on every rank), this rank's slice of row P_n, flags."""
    from . import binding as B

    gamma = logits_shard.shape[1] - 1
    rank = dist.get_rank(group)
    part = B.dssd_edge_partial(logits_shard, draft_tokens, v_begin, temperature)
    ev = B.dssd_edge_combine(all_gather_shards(part["part_ref"], group), all_gather_shards(part["part_sum"], group),
                             all_gather_shards(part["tok_logit"], group), draft_tokens, draft_q_tok, uniforms,
                             temperature, V)
    p_row_shard = B.dssd_edge_emit_shard(logits_shard, ev["accept_len"], ev["row_scale"], temperature)
    mass, ws = B.dssd_resample_shard_mass(p_row_shard, draft_q_shard, ev["accept_len"], gamma)
    draw = B.dssd_resample_shard_draw(all_gather_shards(mass, group), rank, v_begin, p_row_shard, draft_q_shard,
                                      ev["accept_len"], uniforms_rs, gamma, ws)
    token = draw["token"].clone()
    dist.all_reduce(token, op=dist.ReduceOp.MAX, group=group)  # -1 everywhere but on the owning rank
    return {"accept_len": ev["accept_len"], "token": token, "p_row_shard": p_row_shard, "flags": ev["flags"],
            "rs_flags": draw["flags"], "p_tok": ev["p_tok"], "lse": ev["lse"]}

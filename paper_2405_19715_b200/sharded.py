"""Verify/correct across ranks that each hold a slice of the vocabulary (Algorithm 2 of arXiv 2405.19715
under a tensor-parallel output layer): the three local calls of the C ABI with the two all-gathers and
the final reduction between them.  One process per GPU; the exchanges go through `torch.distributed`
(NCCL over NVLink for CUDA tensors) and move B*(K+1)*32 bytes, B*8 bytes and B*4 bytes per rank."""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import specdec as _ops


def vocab_slices(V: int, world: int, multiple: int = 8) -> list[tuple[int, int]]:
    """Contiguous column ranges (offset, size), sizes multiples of `multiple` (16-byte rows) except the last."""
    per = -(-V // world)
    per = -(-per // multiple) * multiple
    out, off = [], 0
    for _ in range(world):
        size = max(0, min(per, V - off))
        out.append((off, size))
        off += size
    if any(sz == 0 for _, sz in out):
        raise ValueError(f"a vocabulary of {V} cannot be split over {world} ranks in multiples of {multiple}")
    return out


def _all_gather(t: torch.Tensor, world: int, group) -> torch.Tensor:
    """[...] on every rank -> [world, ...] in rank order."""
    out = torch.empty((world * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
    dist.all_gather_into_tensor(out, t.contiguous(), group=group)
    return out.view((world,) + tuple(t.shape))


def verify_correct_vocab_sharded(ctx, target_shard, draft_shard, v_offset: int, V: int, cand_tokens, cand_len, uniforms,
                                 temperature: float, group=None, ops=_ops, accept_ratio=None, resid_mass=None):
    """Returns (n_accepted, next_token), identical on every rank of `group`.

    `target_shard` [B, K+1, V_shard] / `draft_shard` [B, K, V_shard] are this rank's columns
    [v_offset, v_offset + V_shard) of the logits; every other argument is replicated.  `ops` supplies the three
    local phases (the CUDA binding unless a test substitutes a model of them)."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    stats = ops.specdec_shard_stats(ctx, target_shard, draft_shard, v_offset, V, cand_tokens, cand_len, temperature)
    stats_all = _all_gather(stats, world, group)
    n_accepted, row_norm, mass = ops.specdec_shard_accept(ctx, target_shard, draft_shard, v_offset, V, stats_all,
                                                          cand_len, uniforms, temperature, accept_ratio=accept_ratio)
    mass_all = _all_gather(mass, world, group)
    next_token = ops.specdec_shard_draw(ctx, target_shard, draft_shard, v_offset, V, stats_all, mass_all, rank,
                                        n_accepted, cand_len, uniforms, row_norm, temperature, resid_mass=resid_mass)
    dist.all_reduce(next_token, op=dist.ReduceOp.MAX, group=group)      # -1 everywhere but on the drawing rank
    return n_accepted, next_token

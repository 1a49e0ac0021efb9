"""Sharding of a batch of sequences over ranks (one process per GPU).

Sequences are independent in the verify-and-feedback step, so rank r of W takes a contiguous
block of sequences and no data crosses ranks on the path.  The only reductions are for reporting:
the slowest rank's time and the number of positions all ranks processed.

The second half of the module is for logits that are sharded along the vocabulary instead (a
tensor-parallel output layer): where the cuts fall, and the three small exchanges between the
phases of the vocabulary-parallel step.  The exchanges move bytes only; all arithmetic on what
they carry happens in the library's kernels.
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_range(B: int, rank: int, world: int) -> Tuple[int, int]:
    """Half-open range [b0, b1) of the sequences of rank ``rank``; sizes differ by at most one."""
    if world < 1 or not (0 <= rank < world) or B < 0:
        raise ValueError("bad rank/world/B")
    base, rem = divmod(B, world)
    b0 = rank * base + min(rank, rem)
    return b0, b0 + base + (1 if rank < rem else 0)


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Largest ``value`` over all ranks (the step time of the job is the slowest rank's)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: str = "cpu") -> float:
    """Sum of ``value`` over all ranks (units processed by the whole job)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def vocab_cuts(V: int, world: int, elem_bytes: int) -> List[Tuple[int, int]]:
    """Half-open column ranges [v0, v1) of the ``world`` shards of a vocabulary of V entries, cut on
    16-byte boundaries (the library's alignment rule); the last shard takes the ragged rest."""
    if world < 1 or V < 1 or elem_bytes not in (2, 4):
        raise ValueError("bad V/world/elem_bytes")
    step = 16 // elem_bytes
    if (V * elem_bytes) % 16 != 0:
        raise ValueError("a row must be a whole number of 16-byte vectors")
    n_vec = V // step
    if n_vec < world:
        raise ValueError("fewer 16-byte vectors in a row than shards")
    base, rem = divmod(n_vec, world)
    cuts, v = [], 0
    for r in range(world):
        w = (base + (1 if r < rem else 0)) * step
        cuts.append((v, v + w))
        v += w
    return cuts


def gather_in_rank_order(local: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather of equally sized tensors: result [world, *local.shape], index = rank."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return local.unsqueeze(0).clone()
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    dist.all_gather([out[r] for r in range(world)], local.contiguous(), group=group)
    return out


def max_of_tokens(tokens: torch.Tensor, group=None) -> torch.Tensor:
    """Element-wise maximum over ranks of the phase-3 token arrays: the owner's token wins over -1."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return tokens
    dist.all_reduce(tokens, op=dist.ReduceOp.MAX, group=group)
    return tokens


def vocab_parallel_step(phases, target_shard, draft_shard, draft_tokens, uniforms, temperature: float,
                        v_offset: int, V_total: int, rank: int, world: int, workspace, group=None):
    """One vocabulary-parallel step of this rank.  ``phases`` supplies the three local calls
    (``partial``, ``finish``, ``draw`` with the binding's signatures); this function only orders them
    and runs the exchanges between them.  Returns (finish outputs, tokens [B,k+1])."""
    records = phases.partial(target_shard, draft_shard, draft_tokens, temperature, v_offset, V_total, workspace)
    all_records = gather_in_rank_order(records, group)
    fin = phases.finish(target_shard, draft_shard, draft_tokens, uniforms, temperature, v_offset, V_total,
                        all_records, world, rank, workspace)
    all_masses = gather_in_rank_order(fin.local_mass, group)
    tokens = phases.draw(target_shard, draft_shard, draft_tokens, uniforms, temperature, v_offset, V_total,
                         fin.accept_len, all_masses, world, rank, fin.status, workspace)
    return fin, max_of_tokens(tokens, group)

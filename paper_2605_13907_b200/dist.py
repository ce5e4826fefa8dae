"""Data-parallel plumbing around the library: which prompts a rank owns, and the one exchange the path needs.

Tokens are independent at the LM head and advantages only couple the G responses of one prompt, so the batch
shards by whole prompts with the LM head replicated.  The only quantity shared by all ranks is the mixing
coefficient alpha: every rank reduces its own rows to the 12 masked sums of ais_diag_moments, the sums are
added over the ranks, and ais_diag_finalize derives the same alpha everywhere.
"""

from __future__ import annotations

import torch
import torch.distributed as dist


def shard_prompts(P: int, world: int, rank: int) -> range:
    """Contiguous block of prompt indices owned by `rank` (sizes differ by at most one)."""
    if not 0 <= rank < world:
        raise ValueError("rank out of range")
    base, extra = divmod(P, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def shard_rows(seq_offsets, G: int, prompts: range):
    """Row range [r0, r1) and local sequence offsets of a block of prompts (sequences of a prompt are consecutive)."""
    s0, s1 = prompts.start * G, prompts.stop * G
    r0, r1 = int(seq_offsets[s0]), int(seq_offsets[s1])
    local = [int(seq_offsets[s]) - r0 for s in range(s0, s1 + 1)]
    return r0, r1, local


def allreduce_moments(moments: torch.Tensor, group=None) -> torch.Tensor:
    """In-place SUM of the moment vector over the ranks of `group` (NCCL for CUDA tensors, gloo for CPU ones)."""
    if moments.dtype != torch.float64:
        raise TypeError("moments must be float64")
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(moments, op=dist.ReduceOp.SUM, group=group)
    return moments

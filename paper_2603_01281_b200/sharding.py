"""Multi-GPU plumbing of the steered-attention path: sequences are independent units.

The path has no exchange step: a sequence (and within it a KV-head group) needs only its own Q, K, V, mask,
gain and routing coefficients, so N ranks take N disjoint sets of sequences and never talk on the data path.
The decode step shards the same way (by sequence), the offline learner by slot (`shard_slots`).
What crosses ranks is bookkeeping only: a barrier around timed regions and the maximum of the ranks' device
times.  These helpers hold that bookkeeping; they work on any torch.distributed backend (NCCL on GPUs, gloo in
the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def shard_sequences(n_sequences: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous range [first, last) of sequence indices owned by `rank`: sizes differ by at most one,
    every sequence has exactly one owner."""
    if world <= 0 or not (0 <= rank < world):
        raise ValueError("bad world/rank: %d/%d" % (world, rank))
    base, extra = divmod(n_sequences, world)
    first = rank * base + min(rank, extra)
    return first, first + base + (1 if rank < extra else 0)


def shard_tokens(cu_seqlens: Sequence[int], world: int, rank: int) -> Tuple[int, int, List[int]]:
    """Token range [t0, t1) of a packed batch owned by `rank`, and the rank's own cu_seqlens (re-based to 0)."""
    first, last = shard_sequences(len(cu_seqlens) - 1, world, rank)
    t0, t1 = int(cu_seqlens[first]), int(cu_seqlens[last])
    return t0, t1, [int(c) - t0 for c in cu_seqlens[first:last + 1]]


def shard_slots(n_slots: int, world: int, rank: int, pair: bool = False) -> Tuple[int, int]:
    """Range [first, last) of (layer, KV head) slots of the offline learner owned by `rank`: slots are learned
    independently (one cross-covariance pair and two SVDs each), so N ranks take N disjoint ranges of the slot axis
    and exchange nothing.  With `pair` (head_dim 64: neighbouring heads share a tensor-core product) the ranges
    start and end on even slots."""
    if pair:
        if n_slots % 2:
            raise ValueError("an even number of slots is needed when heads are processed in pairs")
        first, last = shard_sequences(n_slots // 2, world, rank)
        return 2 * first, 2 * last
    return shard_sequences(n_slots, world, rank)


def rank_seed_offset(rank: int) -> int:
    """Weak scaling: every rank draws its own batch of the same shape; the offset keeps the batches distinct."""
    return int(rank)


def barrier(device_sync=None) -> None:
    """Barrier over the ranks (if a process group is up), then a device synchronise if one is given."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
    if device_sync is not None:
        device_sync()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """The slowest rank's time decides the job's time."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_step: float, steps: int, ms: float, world: int) -> float:
    """Aggregate rate over all ranks: units processed by the whole job per second."""
    return world * units_per_rank_step * steps / (ms * 1e-3)

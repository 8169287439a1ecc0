"""Batch sharding over GPUs: every sequence is independent, so ranks share no data.

Each rank draws its own batch (its seed is a function of the rank) and runs the whole path on its
own GPU; the only communication is the reduction of the timing (max over ranks) and of the byte
count (sum over ranks) that turns per-rank measurements into a whole-job throughput.  There is no
collective on the data path.
"""
from __future__ import annotations


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the batch that `rank` draws: ranks get disjoint, reproducible batches."""
    return int(base_seed) + 1000 * int(rank)


def shard_sequences(n_sequences: int, rank: int, world: int):
    """Contiguous block of sequence indices of `rank` when one batch is split (strong scaling)."""
    per, rem = divmod(int(n_sequences), int(world))
    lo = rank * per + min(rank, rem)
    return lo, lo + per + (1 if rank < rem else 0)


def aggregate(local_ms: float, local_units: float, device=None):
    """(max over ranks of local_ms, sum over ranks of local_units); identity without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_ms), float(local_units)
    dev = device if device is not None else "cpu"
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=dev)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())

"""Host-side plumbing of the N-GPU run: requests are independent (a row reads only its own request's
pages), so the path shards by request with no exchange step.  Every rank draws its own batch of the same
shape (weak scaling); the only communication is a barrier and the reduction of the timing.
"""
from __future__ import annotations


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the batch rank ``rank`` draws: distinct per rank, rank 0 keeps the single-GPU batch."""
    return int(base_seed) + 7919 * int(rank)


def rank_workload(factory, rank: int):
    """The workload of one rank: the named configuration drawn with the rank's own seed."""
    import inspect
    default_seed = inspect.signature(factory).parameters["seed"].default
    return factory(seed=rank_seed(default_seed, rank))


def reduce_job(elapsed_ms: float, units: int, dist=None, device="cpu"):
    """(max over ranks of the elapsed time, sum over ranks of the units processed).

    ``dist`` is ``torch.distributed`` with an initialised default group, or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(elapsed_ms), int(units)
    import torch
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([int(units)], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), int(u.item())

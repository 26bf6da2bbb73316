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


# ---- sharding by KV head -----------------------------------------------------------------------------------------
# The second natural cut of the path: a query head reads only its own KV head, so rank r of N can own KV heads
# [r * Hkv / N, (r + 1) * Hkv / N), the query heads of those groups and the page pools of those heads.  Every rank sees
# the same batch of DAGs (the planner's input and its canonical tables do not change; only the head count the work lists
# are cut for does), runs the library on its slice, and the output is the concatenation of the ranks' slices along the
# head axis.  There is no exchange step inside the path: the all-gather of the output below stands outside it (what
# follows attention in a model, the output projection, can equally consume the slices where they are).

def head_slice(n_q_heads: int, n_kv_heads: int, rank: int, world: int):
    """(first query head, query heads, first KV head, KV heads) of rank ``rank`` when the KV heads are dealt out evenly."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("rank / world")
    if n_kv_heads % world != 0 or n_q_heads % n_kv_heads != 0:
        raise ValueError(f"{n_kv_heads} KV heads cannot be dealt out evenly over {world} ranks")
    group = n_q_heads // n_kv_heads
    kv_per = n_kv_heads // world
    return rank * kv_per * group, kv_per * group, rank * kv_per, kv_per


def slice_heads(x, first: int, count: int):
    """The head slice [first, first + count) of a [tokens, heads, head_dim] array or tensor, contiguous."""
    y = x[:, first:first + count]
    return y.contiguous() if hasattr(y, "contiguous") else y.copy()


def gather_heads(out_slice, dist=None):
    """All ranks' output slices [rows, heads / N, head_dim] put together along the head axis: [rows, heads, head_dim] on
    every rank (torch tensors; NCCL on GPUs, gloo on CPU).  A single process returns its slice."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return out_slice
    import torch
    parts = [torch.empty_like(out_slice) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, out_slice.contiguous())
    return torch.cat(parts, dim=1)

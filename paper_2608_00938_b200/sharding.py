"""Multi-GPU plumbing: the decode path shards by request and has no data-path collective.

Beams interact only inside a request (top-k, matcher and encoder K/V are per request), so ranks
own disjoint request ranges and replicate the trie and the weights.  The only cross-rank traffic is
timing (max over ranks) and, optionally, gathering the small per-request results.
"""
from __future__ import annotations


def request_shard(n_requests: int, world: int, rank: int) -> range:
    """Contiguous, balanced range of request ids owned by `rank` (sizes differ by at most one)."""
    base, extra = divmod(n_requests, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank scalar (e.g. a device-timed duration) over the default process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_results(local, device=None):
    """All-gather of equally shaped per-rank result tensors (scores / keys of the final beams)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [local]
    out = [torch.empty_like(local) for _ in range(dist.get_world_size())]
    dist.all_gather(out, local)
    return out

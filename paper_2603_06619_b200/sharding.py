"""Data-parallel sharding of the path: host-side logic only.

Responses are independent given the global batch size B, and advantages need
only the G responses of one prompt, so ranks take whole prompt groups.  With
the GLOBAL B in every rank's loss parameters the job's loss and dW are the sums
of the ranks' losses and dW (one all-reduce in a trainer; none is needed for
the selection, whose draws are keyed by the GLOBAL response index).
"""
import torch
import torch.distributed as dist


def prompt_range(P, rank, world):
    """Contiguous block of prompts [lo, hi) owned by `rank` (sizes differ by at most one)."""
    base, extra = divmod(P, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def response_range(P, G, rank, world):
    lo, hi = prompt_range(P, rank, world)
    return lo * G, hi * G


def rank_seed(seed, rank):
    """Seed of the independent batch a rank draws in the weak-scaling benchmark."""
    return seed + rank


def aggregate_timing(elapsed_ms, units, device=None):
    """(max over ranks of each elapsed time, sum over ranks of the units processed).

    `elapsed_ms` is a list of floats measured on this rank; every rank gets the result.
    """
    t = torch.tensor(list(elapsed_ms), dtype=torch.float64, device=device)
    n = torch.tensor([float(units)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], float(n.item())

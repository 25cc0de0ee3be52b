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


def allreduce_grads(loss, dW, bucket_elems=64 << 20, wait=True):
    """Sum `loss` (1 element) and `dW` ([V, d] float32) over the data-parallel ranks, in place.

    This is the one exchange of a data-parallel step: every rank computed its responses'
    share with the GLOBAL batch size in its weights, so the sums are the job's loss and
    gradient.  dW goes out in buckets (one collective each, issued asynchronously on the
    process group's stream) so that a caller that passes wait=False can overlap the tail of
    its own work with them; it gets the handles to wait on.  A single process is a no-op.
    """
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return []
    flat = dW.reshape(-1)
    handles = [dist.all_reduce(flat[lo:lo + bucket_elems], async_op=True)
               for lo in range(0, flat.numel(), bucket_elems)]
    handles.append(dist.all_reduce(loss, async_op=True))
    if wait:
        for h in handles:
            h.wait()
        return []
    return handles


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

"""Multi-GPU use of the path: heads are independent, so a job shards the B*H heads (or the batch) across
ranks and every rank runs the single-GPU library on its slice.  There is no exchange step and no collective
in the data path; only timing (max over ranks) and reporting cross ranks."""


def head_range(total_heads, rank, world_size):
    """Contiguous, balanced slice [lo, hi) of `total_heads` flat head indices (b * H + h) owned by `rank`.
    The first `total_heads % world_size` ranks get one head more."""
    if world_size <= 0 or not 0 <= rank < world_size or total_heads < 0:
        raise ValueError("bad rank / world_size / total_heads")
    base, extra = divmod(total_heads, world_size)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(value, dist=None, device=None):
    """Max of a python float over all ranks (the time of a multi-GPU step is its slowest rank's)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())

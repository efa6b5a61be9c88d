"""Rank bookkeeping for runs on several GPUs.

(batch, head) pairs of the operator are independent problems, so several GPUs simply take different
batches: there is no collective on the data path.  What remains is host logic, kept here so that it
can be exercised with CPU ranks: which seed a rank draws its batch from, which slice of a global
batch it owns, and how per-rank timings and unit counts combine into one job-wide figure (slowest
rank's time, sum of units).  Works with any initialised ``torch.distributed`` backend.
"""
import os


def rank_env():
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) without one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_seed(base_seed, rank):
    """Seed of a rank's own synthetic batch: distinct per rank, rank 0 reproduces the 1-GPU run."""
    return int(base_seed) + int(rank)


def batch_slice(global_batch, rank, world):
    """Contiguous slice [lo, hi) of a global batch owned by `rank`; sizes differ by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank %d outside world of %d" % (rank, world))
    base, extra = divmod(int(global_batch), int(world))
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def aggregate(ms_local, units_local, device="cpu"):
    """Job-wide (time, units): max of the ranks' times and sum of their units.

    Without an initialised process group the local values are returned unchanged.
    """
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), int(units_local)
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    u = torch.tensor([int(units_local)], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), int(u.item())


def throughput(units_total, ms_max):
    """Units per second of the whole job."""
    return units_total / (ms_max * 1e-3)

"""Host-side bookkeeping for running independent replicas, one process per GPU.

The SOAP path has no exchange step: a centre needs only the atoms inside its own cutoff sphere,
so several GPUs simply work on their own structures.  The only communication is for measurement:
a barrier and a maximum over ranks of the timed durations (torch.distributed; NCCL on GPUs, gloo in
the CPU tests)."""
from __future__ import annotations


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def job_throughput(units_per_rank: int, world_size: int, slowest_ms: float) -> float:
    """Units per second of the whole job when every rank processes `units_per_rank` units and the
    slowest rank needs `slowest_ms` for them (weak scaling)."""
    return world_size * units_per_rank / (slowest_ms * 1e-3)


def split_centers(n_centers: int, world_size: int, rank: int):
    """Contiguous, near-equal range of centre indices for `rank`: how `bench.py --shard` cuts one structure
    into one piece per GPU (a centre needs only the atoms inside its sphere, so nothing is exchanged)."""
    base, extra = divmod(n_centers, world_size)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)

"""Multi-GPU plumbing for the decode path: one process per GPU, batch-sharded.

Every (batch item, kv head) of the decode problem is independent (the paper lifts the
single-head computation over leading batch/head indices), so sharding the batch over ranks
needs no data-path collective: each rank owns a contiguous slice of q / K / V / out.  The
only communication is control-plane: a barrier around timed regions, a MAX reduction of the
per-rank step time and a SUM of the bytes processed.  Works with any torch.distributed
backend (NCCL on GPUs, gloo in CPU tests).
"""
from __future__ import annotations


def shard_batch(global_batch: int, world: int, rank: int):
    """Contiguous slice [start, start+count) of the batch owned by `rank`: the first
    `global_batch % world` ranks get one extra item; ranks beyond the batch get count 0."""
    if global_batch < 0 or world < 1 or not (0 <= rank < world):
        raise ValueError("bad shard arguments")
    base, extra = divmod(global_batch, world)
    count = base + (1 if rank < extra else 0)
    start = rank * base + min(rank, extra)
    return start, count


def reduce_step_time(ms_local: float, device="cpu") -> float:
    """Step time of the whole job = the slowest rank's (MAX over ranks)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(ms_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def reduce_sum(x: float, device="cpu") -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput_gbs(bytes_local: float, ms_local: float, device="cpu") -> float:
    """Whole-job GB/s: bytes summed over ranks / the slowest rank's time."""
    total = reduce_sum(bytes_local, device)
    ms = reduce_step_time(ms_local, device)
    return total / (ms * 1e-3) / 1e9


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()

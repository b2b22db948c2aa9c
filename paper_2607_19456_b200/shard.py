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


# ---- sequence split: one long sequence over several GPUs --------------------------------
# Each rank holds a contiguous range of cached rows of every (batch, kv head) and computes
# the unnormalised triple (o, m, l) over it (moa_decode_attn_partial); one all-gather of
# batch * h_q * (d_v + 4) floats per rank is the only exchange, after which every rank
# merges the triples in rank order (moa_combine_partials).  The exchange goes through the
# process group (NCCL over NVLink on GPUs, gloo in CPU tests): remote triples land in local
# memory first, no kernel reads a peer's memory.

def shard_rows(n: int, world: int, rank: int, align: int = 16):
    """Contiguous row range [start, start+count) owned by `rank` when n cached rows are cut
    into `world` ranges whose sizes are multiples of `align` (except the last non-empty
    one).  Ranks past the end of the sequence get count 0."""
    if n < 0 or world < 1 or not (0 <= rank < world) or align < 1:
        raise ValueError("bad shard arguments")
    per = -(-n // world)
    per = -(-per // align) * align
    start = min(n, rank * per)
    return start, min(n, start + per) - start


def empty_partial(batch: int, h_q: int, d_v: int, like=None):
    """The triple of an empty row range: o = 0, m = -inf, l = 0 (ignored by the merge)."""
    import torch
    t = torch.zeros((batch, h_q, d_v + 4), dtype=torch.float32,
                    device=like.device if like is not None else "cpu")
    t[:, :, d_v] = float("-inf")
    return t


def gather_partials(partial_local, group=None):
    """All-gather the per-rank triples [batch, h_q, d_v+4] into [world, batch, h_q, d_v+4],
    ordered by rank.  Without an initialised process group: a world of one."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return partial_local.unsqueeze(0).contiguous()
    world = dist.get_world_size(group)
    parts = [torch.empty_like(partial_local) for _ in range(world)]
    dist.all_gather(parts, partial_local.contiguous(), group=group)
    return torch.stack(parts, dim=0)


def seq_split_decode(q, K_rows, V_rows, out, scale: float, group=None):
    """Decode attention when every rank holds a row range of the same sequences.
    q [batch, h_q, d_k] (replicated), K_rows / V_rows [batch, h_kv, n_local, d] on this
    rank's GPU (n_local may be 0), out [batch, h_q, d_v] (every rank gets the result)."""
    import paper_2607_19456_b200 as moa
    batch, h_q, d_k = q.shape
    h_kv, n_local, d_v = K_rows.shape[1], K_rows.shape[2], V_rows.shape[3]
    if n_local > 0:
        import torch
        part = torch.empty((batch, h_q, d_v + 4), dtype=torch.float32, device=q.device)
        moa.moa_decode_attn_partial(q, K_rows, V_rows, part, batch, h_q, h_kv, n_local, d_k, d_v, scale)
    else:
        part = empty_partial(batch, h_q, d_v, like=q)
    parts = gather_partials(part, group)
    moa.moa_combine_partials(parts, parts.shape[0], out, batch, h_q, d_v)
    return out

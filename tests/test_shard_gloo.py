"""The N > 1 path on CPU: two gloo ranks each own a batch shard (no data-path collective),
their outputs concatenate to the unsharded result, and the timing / throughput reductions
are MAX / SUM over ranks.  The oracle stands in for the GPU kernels here."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, global_batch, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import moa_inputs as mi
        import oracle
        from paper_2607_19456_b200 import shard
        w = mi.Workload("sh", 77, global_batch, 8, 2, 40, 16, 16)
        start, count = shard.shard_batch(global_batch, world, rank)
        qq, K, V = w.q(), w.K(), w.V()
        mine = oracle.decode(qq[start:start + count], K[start:start + count], V[start:start + count],
                             w.scale) if count else np.zeros((0, 8, 16), np.float32)
        shard.barrier()
        parts = [None] * world
        dist.all_gather_object(parts, (start, mine))
        ms = shard.reduce_step_time(10.0 * (rank + 1))
        gbs = shard.job_throughput_gbs(1e9 * (rank + 1), 10.0 * (rank + 1))
        if rank == 0:
            full = np.concatenate([p[1] for p in sorted(parts, key=lambda t: t[0])], axis=0)
            q.put((full, ms, gbs))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("global_batch", [5, 2])
def test_two_ranks_batch_sharded(global_batch):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, global_batch, q)) for r in range(2)]
    for p in procs:
        p.start()
    full, ms, gbs = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sys.path.insert(0, ROOT)
    import moa_inputs as mi
    import oracle
    w = mi.Workload("sh", 77, global_batch, 8, 2, 40, 16, 16)
    assert np.array_equal(full, oracle.decode(w.q(), w.K(), w.V(), w.scale))
    assert ms == 20.0                                   # MAX over ranks
    assert abs(gbs - 3e9 / 20e-3 / 1e9) < 1e-9          # SUM of bytes / slowest time


def test_shard_batch_covers_the_batch_exactly_once():
    from paper_2607_19456_b200.shard import shard_batch
    for B in (0, 1, 5, 16, 33):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                s, c = shard_batch(B, world, r)
                seen += list(range(s, s + c))
            assert seen == list(range(B))
            sizes = [shard_batch(B, world, r)[1] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_batch(4, 2, 2)


# ---- sequence split: every rank holds a row range, one all-gather of (o, m, l) triples ----
def _numpy_partial(q, K, V, scale):
    """Unnormalised triple over the given rows, in fp64, log2 domain (test code)."""
    B, hq, _ = q.shape
    hkv, n, dv = K.shape[1], K.shape[2], V.shape[3]
    out = np.zeros((B, hq, dv + 4), np.float32)
    out[:, :, dv] = -np.inf
    if n == 0:
        return out
    gs = hq // hkv
    for b in range(B):
        for g in range(hq):
            s2 = (K[b, g // gs].astype(np.float64) @ q[b, g].astype(np.float64)) * scale * np.log2(np.e)
            m = s2.max()
            w = np.exp2(s2 - m)
            out[b, g, :dv] = w @ V[b, g // gs].astype(np.float64)
            out[b, g, dv], out[b, g, dv + 1] = m, w.sum()
    return out


def _numpy_combine(parts, dv):
    m = parts[..., dv].astype(np.float64)
    M = m.max(axis=0)
    f = np.where(np.isneginf(m), 0.0, np.exp2(m - M))
    L = (parts[..., dv + 1] * f).sum(axis=0)
    return ((parts[..., :dv] * f[..., None]).sum(axis=0) / L[..., None]).astype(np.float32)


def _seq_worker(rank, world, port, n, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import moa_inputs as mi
        from paper_2607_19456_b200 import shard
        w = mi.Workload("sq", 91, 2, 8, 2, n, 16, 16)
        qq, K, V = w.q(), w.K(), w.V()
        start, count = shard.shard_rows(n, world, rank)
        part = torch.from_numpy(_numpy_partial(qq, K[:, :, start:start + count], V[:, :, start:start + count], w.scale))
        if count == 0:
            assert torch.equal(part, shard.empty_partial(2, 8, 16))
        parts = shard.gather_partials(part)
        assert parts.shape == (world, 2, 8, 20)
        assert torch.equal(parts[rank], part)          # rank order
        if rank == 0:
            q.put(_numpy_combine(parts.numpy(), 16))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("n", [100, 16, 5])
def test_two_ranks_sequence_split(n):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_seq_worker, args=(r, 2, port, n, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sys.path.insert(0, ROOT)
    import moa_inputs as mi
    import oracle
    w = mi.Workload("sq", 91, 2, 8, 2, n, 16, 16)
    assert float(np.max(np.abs(got - oracle.decode(w.q(), w.K(), w.V(), w.scale)))) <= 1e-6


def test_shard_rows_covers_the_sequence_exactly_once():
    from paper_2607_19456_b200.shard import shard_rows
    for n in (0, 1, 15, 16, 17, 100, 4096, 4097):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                s, c = shard_rows(n, world, r)
                assert c >= 0 and (c % 16 == 0 or s + c == n)
                seen += list(range(s, s + c))
            assert seen == list(range(n))

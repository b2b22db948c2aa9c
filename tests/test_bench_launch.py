"""bench.py's own multi-rank launch path, on CPU: the environment it builds for its child
ranks, and the whole timing / reduction loop of two gloo ranks with the oracle standing in
for the kernels (batch shard: no data-path collective, MAX over ranks of the step time)."""
import io
import json
import os
import sys
from contextlib import redirect_stdout

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def test_child_rank_environment():
    base = {"PATH": "/bin", "WORLD_SIZE": "7"}
    envs = [bench.rank_env(r, 2, 29871, base) for r in range(2)]
    for r, e in enumerate(envs):
        assert e["RANK"] == str(r) and e["LOCAL_RANK"] == str(r) and e["WORLD_SIZE"] == "2"
        assert e["MASTER_ADDR"] == "127.0.0.1" and e["MASTER_PORT"] == "29871"
        assert e["PATH"] == "/bin"
    assert base["WORLD_SIZE"] == "7"                      # the caller's environment is not touched


def test_gpus_flag_spawns_only_without_a_launcher(monkeypatch):
    calls = []
    monkeypatch.setattr(bench, "spawn_ranks", lambda world, argv: calls.append((world, list(argv))) or 0)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    assert bench.main(["--gpus", "2", "--steps", "4"]) == 0
    assert calls == [(2, ["--gpus", "2", "--steps", "4"])]


class OracleStandIn:
    """What bench.py times, with the CPU oracle in place of the CUDA library (tests only)."""

    def __init__(self, w, rank, world):
        import oracle
        self.oracle, self.w = oracle, w
        self.q, self.K, self.V = w.q(), w.K(), w.V()
        self.decode_bytes = oracle.min_bytes(w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v)
        self.bytes_per_step = self.decode_bytes
        self.l2_note = "host memory"
        self.steps_run = 0

    def step(self):
        self.out = self.oracle.decode(self.q, self.K, self.V, self.w.scale)
        self.steps_run += 1

    def reset(self):
        pass

    def profile(self, mode):
        self.mark = self.steps_run

    def profile_read(self):
        return 0.0, 0, self.steps_run - self.mark


def _rank(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(bench.rank_env(rank, world, port))
    args = bench.parse_args(["--gpus", str(world), "--steps", "5", "--warmup", "3", "--workload", "single_head",
                             "--no-others", "--no-cpu", "--e2e-steps", "0"])
    buf = io.StringIO()
    with redirect_stdout(buf):
        bench.run_rank(args, bench.HostSide(), make_run=OracleStandIn)
    q.put((rank, buf.getvalue()))


def test_two_gloo_ranks_run_the_whole_bench_loop():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = bench.free_port()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[1].strip() == ""                            # only rank 0 prints
    line = json.loads(got[0].strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["steps"] == 5 and line["scaling"] == "weak"
    assert len(line["us_per_step_per_rank"]) == 2
    assert abs(line["us_per_step"] - max(line["us_per_step_per_rank"])) < 1e-6
    w = bench.mi.WORKLOADS["single_head"]
    per_rank = 4 * (w.batch * w.h_kv * w.n * (w.d_k + w.d_v) + w.batch * w.h_q * (w.d_k + w.d_v))
    assert np.isclose(line["value"], 2 * per_rank / (line["ms_per_step"] * 1e-3) / 1e9)
    assert line["gpu_launches"] == 5 and line["roofline"] is None

#!/usr/bin/env python
"""Benchmark of the decode-attention hot path (libmoa) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one pass of the whole hot path over one batch of synthetic input: the
KV-cache append of the new token's (k, v) row followed by decode attention over the
cache (for the multi-step workload: one fused append+attend step over ragged lengths).
Prints ONE JSON line (rank 0).  `value` is the achieved algorithmic HBM bandwidth of the
whole job (bytes of the paper's traffic model per step, summed over ranks, divided by
the step time, max over ranks); `ms_per_step` is the step time.

With N > 1 every rank (one per GPU) runs its own shard of an N-times larger batch: the path
has no exchange step, so there is no data-path collective and the scaling is weak.  Under
torchrun the ranks are the launcher's; started plainly with `--gpus N`, this script starts
the N ranks itself (one child process per GPU, rendezvous on 127.0.0.1).  `--split seq`
instead cuts the cached rows of one workload over the ranks (one all-gather of the partial
triples per step; strong scaling).

`--impl reference` times the plain CPU oracle (the only reference there is for this
paper) on a bounded sample of the same workload, on the host cores.
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import moa_inputs as mi  # noqa: E402

METRIC = "decode-attention achieved HBM GB/s (algorithmic bytes per step / step time; us/step = 1000*ms_per_step)"
UNIT = "GB/s"
DEFAULT_WORKLOAD = "gqa"
FALLBACK_HBM_GBS = 6650.0
L2_BYTES_ASSUMED = 126 * 1024 * 1024

# DRAM traffic of one launch of the dominant kernel, from an ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum), per workload.  Every entry is stamped with
# a digest of the kernel sources it was captured with; when those files have changed since,
# the figure is stale and the line reports null instead.
NCU_TRAFFIC = {
    "gqa": {"bytes": 1074629632 + 1160704, "sources": ["moa_stream.cuh", "moa_device.cuh"], "digest": "5eab75429bf75dce"},
    "extra_group8_d128": {"bytes": 1075606784 + 769792, "sources": ["moa_mma.cuh", "moa_device.cuh"], "digest": "7c7e6fb243ebb37f"},
    "multi_step": {"bytes": 351830272 + 909056, "sources": ["moa_stream.cuh", "moa_device.cuh"], "digest": "5eab75429bf75dce"},
    "mqa_long": {"bytes": 537116160 + 265472, "sources": ["moa_grouped64.cuh", "moa_grouped.cuh", "moa_tc.cuh"], "digest": "d68ab0582bbd0527"},
    "extra_mqa_d64": {"bytes": 537045504 + 388608, "sources": ["moa_grouped64.cuh", "moa_grouped.cuh", "moa_tc.cuh"], "digest": "d68ab0582bbd0527"},
}


def source_digest(files):
    import hashlib
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_2607_19456_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(wname):
    e = NCU_TRAFFIC.get(wname)
    if not e:
        return None
    try:
        return e["bytes"] if source_digest(e["sources"]) == e["digest"] else None
    except OSError:
        return None


def env_int(name, default):
    try:
        return int(os.environ.get(name, default))
    except ValueError:
        return default


def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------------------
# clocks sampled during the timed region (NVML, read-only)
# --------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
               0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x100: "display_clock_setting"}

    def __init__(self, index, interval=0.02):
        # NVML queries go through the driver; polling them every couple of milliseconds
        # measurably slows the kernels being timed, so sample sparsely.
        self.interval = interval
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = self._handle(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _handle(self, index):
        import torch
        try:
            uuid = str(torch.cuda.get_device_properties(index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            return self.nv.nvmlDeviceGetHandleByUUID(uuid)
        except Exception:
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(vis.split(",")[index]) if vis and vis.split(",")[index].isdigit() else index
            return self.nv.nvmlDeviceGetHandleByIndex(phys)

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for bit, name in self.REASONS.items():
                    if r & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.interval)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "samples": len(self.samples),
                "reasons": sorted(self.reasons)}


# --------------------------------------------------------------------------------------
# workloads on the device
# --------------------------------------------------------------------------------------
def pinned_like(shape):
    import torch
    return torch.empty(shape, dtype=torch.float32, pin_memory=True)


# Shapes outside the five benchmark configurations, timed only, to show the kernels that
# those five do not reach: groups of 8 and 16 heads (warp-MMA streaming kernel) and d = 32.
EXTRA_WORKLOADS = {
    "extra_group8_d128": mi.Workload("extra_group8_d128", 1101, 16, 64, 8, 8192, 128, 128),
    "extra_group8_d64": mi.Workload("extra_group8_d64", 1102, 16, 64, 8, 16384, 64, 64),
    "extra_group16_d128": mi.Workload("extra_group16_d128", 1103, 16, 128, 8, 8192, 128, 128),
    "extra_mha_d32": mi.Workload("extra_mha_d32", 1104, 64, 32, 32, 4096, 32, 32),
    # 32 query heads on one K/V head at d = 64 (the shape of the paper's GQA/MQA traffic table), long cache
    "extra_mqa_d64": mi.Workload("extra_mqa_d64", 1105, 8, 32, 1, 131072, 64, 64),
}
# Workloads whose step is issued as two calls, moa_kv_append + moa_decode_attn, instead of the
# fused moa_append_decode (none at present; kept for A/B timing of the two forms).
TWO_CALL_STEP = set()


class DenseRun:
    """append one row at the last position, then decode over n rows (dense cache)."""

    def __init__(self, w, seed_shift=0, host_inputs=True, device="cuda"):
        import torch
        import paper_2607_19456_b200 as moa
        self.moa, self.torch, self.w = moa, torch, w
        B, hq, hkv, n, dk, dv = w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v
        self.bytes_per_step = moa.moa_min_bytes(B, hq, hkv, n, dk, dv) + 2 * B * hkv * (dk + dv) * 4
        self.decode_bytes = moa.moa_min_bytes(B, hq, hkv, n, dk, dv)
        one = self.decode_bytes
        # consecutive steps never touch the same buffers: at least two independent sets, and as
        # many as it takes to exceed twice the L2 size
        self.nsets = max(2, min(4096, -(-2 * L2_BYTES_ASSUMED // one)))
        S = self.nsets
        ws = mi.small_like(w, seed=w.seed + seed_shift)
        self.host = None
        if host_inputs:
            self.host = dict(q=pinned_like((B, hq, dk)), K=pinned_like((B, hkv, n, dk)),
                             V=pinned_like((B, hkv, n, dv)), out=pinned_like((B, hq, dv)))
            ws.q(out=self.host["q"].numpy())
            ws.K(out=self.host["K"].numpy())
            ws.V(out=self.host["V"].numpy())
            self.k_new_h = mi.normal(ws.seed, mi.TID_KNEW, (B, hkv, dk))
            self.v_new_h = mi.normal(ws.seed, mi.TID_VNEW, (B, hkv, dv))
            self.q = torch.empty((S, B, hq, dk), device=device)
            self.K = torch.empty((S, B, hkv, n, dk), device=device)
            self.V = torch.empty((S, B, hkv, n, dv), device=device)
            for s in range(S):
                self.q[s].copy_(self.host["q"]); self.K[s].copy_(self.host["K"]); self.V[s].copy_(self.host["V"])
            self.k_new = torch.from_numpy(self.k_new_h).to(device)
            self.v_new = torch.from_numpy(self.v_new_h).to(device)
        else:
            g = torch.Generator(device=device).manual_seed(ws.seed)
            self.q = torch.randn((S, B, hq, dk), device=device, generator=g)
            self.K = torch.randn((S, B, hkv, n, dk), device=device, generator=g)
            self.V = torch.randn((S, B, hkv, n, dv), device=device, generator=g)
            if w.v_dist == "uniform":
                self.V.uniform_(-1, 1, generator=g)
            self.k_new = torch.randn((B, hkv, dk), device=device, generator=g)
            self.v_new = torch.randn((B, hkv, dv), device=device, generator=g)
        self.out = torch.zeros((S, B, hq, dv), device=device)
        self.pos = torch.full((B,), n - 1, dtype=torch.int32, device=device)
        self.i = 0
        # raw addresses, so that the timed loop does no tensor indexing on the host
        self.ptrs = [(self.q[s].data_ptr(), self.K[s].data_ptr(), self.V[s].data_ptr(),
                      self.out[s].data_ptr()) for s in range(S)]
        self.aux = (self.k_new.data_ptr(), self.v_new.data_ptr(), self.pos.data_ptr())
        self.ws_bytes = moa.moa_workspace_bytes(B, hq, hkv, n, dk, dv)
        self.wsbuf = torch.empty(self.ws_bytes, dtype=torch.uint8, device=device)
        self.wsptr = self.wsbuf.data_ptr()
        self.stream = torch.cuda.current_stream().cuda_stream
        self.two_call = w.name in TWO_CALL_STEP
        self.l2_note = "rotating over %d buffer sets of %.0f MB (%.0f MB in total; L2 is 126 MB)" % (S, one / 1e6, S * one / 1e6)

    def step(self):
        w, m = self.w, self.moa
        q, K, V, out = self.ptrs[self.i % self.nsets]
        kn, vn, pos = self.aux
        self.i += 1
        if self.two_call:
            m.moa_kv_append(K, V, kn, vn, pos, w.batch, w.h_kv, w.n, w.d_k, w.d_v, self.stream)
            m.moa_decode_attn(q, K, V, out, w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale, self.stream)
            return
        m.moa_append_decode(q, K, V, kn, vn, out, pos, w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale,
                            self.wsptr, self.ws_bytes, self.stream)

    def reset(self):
        self.i = 0

    def profile(self, mode):
        self.moa.moa_profile(mode)

    def profile_read(self):
        return self.moa.moa_profile_read()

    def e2e_step(self):
        w, h = self.w, self.host
        self.moa.moa_decode_attn_host(h["q"], h["K"], h["V"], h["out"], w.batch, w.h_q, w.h_kv, w.n,
                                      w.d_k, w.d_v, w.scale)
        return float(h["out"][0, 0, 0])

    def e2e_bytes(self):
        h = self.host
        return (sum(h[k].numel() * 4 for k in ("q", "K", "V")), h["out"].numel() * 4)

    def resident_step(self):
        """A step as a serving loop sees it: the cache stays on the device; the token's q, k, v
        come from pinned host memory, the output goes back to pinned host memory."""
        w, h, t = self.w, self.host, self.torch
        if not hasattr(self, "res"):
            self.res = dict(k=pinned_like(self.k_new.shape), v=pinned_like(self.v_new.shape))
            self.res["k"].copy_(self.k_new); self.res["v"].copy_(self.v_new)
        self.q[0].copy_(h["q"], non_blocking=True)
        self.k_new.copy_(self.res["k"], non_blocking=True)
        self.v_new.copy_(self.res["v"], non_blocking=True)
        q, K, V, out = self.ptrs[0]
        kn, vn, pos = self.aux
        self.moa.moa_append_decode(q, K, V, kn, vn, out, pos, w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale,
                                   self.wsptr, self.ws_bytes, self.stream)
        h["out"].copy_(self.out[0], non_blocking=True)
        t.cuda.synchronize()
        return float(h["out"][0, 0, 0])


class MultiStepRun:
    """ragged multi-step decode: fused append + attend + length advance per step."""

    def __init__(self, w, seed_shift=0, device="cuda", host_inputs=True):
        import torch
        import paper_2607_19456_b200 as moa
        self.moa, self.torch, self.w = moa, torch, w
        B, hq, hkv, n_max, dk, dv, T = w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.steps
        ws = mi.small_like(w, seed=w.seed + seed_shift)
        self.lens0_h = ws.start_lens()
        K = ws.K(); V = ws.V()
        for b in range(B):
            K[b, :, self.lens0_h[b]:] = 0
            V[b, :, self.lens0_h[b]:] = 0
        self.K, self.V = torch.from_numpy(K).to(device), torch.from_numpy(V).to(device)
        self.host = dict(K=K, V=V)
        self.k_new = torch.from_numpy(mi.normal(ws.seed, mi.TID_KNEW, (T, B, hkv, dk))).to(device)
        self.v_new = torch.from_numpy(mi.normal(ws.seed, mi.TID_VNEW, (T, B, hkv, dv))).to(device)
        self.q = torch.from_numpy(mi.normal(ws.seed, mi.TID_QSTEP, (T, B, hq, dk))).to(device)
        self.out = torch.zeros((B, hq, dv), device=device)
        self.lens0 = torch.from_numpy(self.lens0_h).to(device)
        self.lens = self.lens0.clone()
        self.ws_bytes = moa.moa_workspace_bytes(B, hq, hkv, n_max, dk, dv)
        self.wsbuf = torch.empty(self.ws_bytes, dtype=torch.uint8, device=device)
        self.t = 0
        self.nsets = 1
        self.step_ptrs = [(self.q[t].data_ptr(), self.k_new[t].data_ptr(), self.v_new[t].data_ptr())
                          for t in range(T)]
        self.fix_ptrs = (self.K.data_ptr(), self.V.data_ptr(), self.out.data_ptr(), self.lens.data_ptr(),
                         self.wsbuf.data_ptr())
        self.stream = torch.cuda.current_stream().cuda_stream
        self.l2_note = "every step streams the whole live cache (about 400 MB, larger than L2)"

    def bytes_for_steps(self, t0, t1):
        w = self.w
        tot = 0
        for t in range(t0, t1):
            rows = int((self.lens0_h.astype(np.int64) + t + 1).sum())
            tot += (w.h_kv * rows * (w.d_k + w.d_v) + w.batch * w.h_q * (w.d_k + w.d_v)
                    + 2 * w.batch * w.h_kv * (w.d_k + w.d_v)) * 4
        return tot

    def step(self):
        w, m, t = self.w, self.moa, self.t
        if t >= w.steps:
            raise RuntimeError("multi_step: warmup + steps must not exceed %d" % w.steps)
        q, kn, vn = self.step_ptrs[t]
        K, V, out, lens, wsb = self.fix_ptrs
        m.moa_decode_step(q, K, V, kn, vn, out, lens, w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale,
                          wsb, self.ws_bytes, self.stream)
        self.t += 1

    def reset(self):
        self.lens.copy_(self.lens0)
        self.t = 0

    def profile(self, mode):
        self.moa.moa_profile(mode)

    def profile_read(self):
        return self.moa.moa_profile_read()


class CudaSide:
    """Where the steps run and how they are timed: one GPU, CUDA events on the current stream."""
    backend, device = "nccl", "cuda"

    def __init__(self, local):
        import torch
        self.torch = torch
        torch.cuda.set_device(local)

    def sync(self):
        self.torch.cuda.synchronize()

    def mark(self):
        e = self.torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    @staticmethod
    def ms_between(e0, e1):
        return e0.elapsed_time(e1)


class HostSide:
    """The same protocol without a GPU (gloo ranks, wall clock): it exists so that the launch
    and reduction path of N ranks can be exercised on a CPU-only machine with a stand-in
    for the kernels; bench.py itself never selects it."""
    backend, device = "gloo", "cpu"

    def sync(self):
        pass

    def mark(self):
        return time.perf_counter()

    @staticmethod
    def ms_between(e0, e1):
        return (e1 - e0) * 1e3


def time_steps(run, steps, warmup, side, sampler=None, bracket=False, segment=0):
    """-> (ms per step, decode-kernel ms per launch or None, launches in the timed region, clocks,
    [ms per step of the first and of the last `segment` steps] or None).
    With bracket=True the library also records a CUDA event pair around every launch of
    the dominant decode kernel (which costs a few microseconds per launch)."""
    run.reset()
    for _ in range(warmup):
        run.step()
    side.sync()
    if isinstance(run, MultiStepRun):
        run.reset()
    barrier()
    side.sync()
    if sampler:
        sampler.start()
    run.profile(2 if bracket else 1)
    have_segs = 0 < segment and 2 * segment <= steps
    cuts = sorted({0, steps} | ({segment, steps - segment} if have_segs else set()))
    marks = {}
    for i in range(steps + 1):
        if i in cuts:
            marks[i] = side.mark()
        if i < steps:
            run.step()
    side.sync()
    kern_ms, kern_n, launches = run.profile_read()
    LAST_BRACKETED.clear()
    if bracket and kern_n:
        LAST_BRACKETED.extend(run.moa.moa_profile_launch_ms(i) * 1e3 for i in range(int(kern_n)))
    run.profile(0)
    clocks = sampler.stop() if sampler else None
    barrier()
    ms = side.ms_between(marks[0], marks[steps]) / steps
    segs = None
    if have_segs:
        segs = [side.ms_between(marks[0], marks[segment]) / segment,
                side.ms_between(marks[steps - segment], marks[steps]) / segment]
    return ms, (kern_ms / kern_n if kern_n else None), launches, clocks, segs


_DIST = {"on": False, "device": "cuda"}
LAST_BRACKETED = []      # per-launch event times (us) of the last bracketed pass


def barrier():
    if _DIST["on"]:
        from paper_2607_19456_b200 import shard
        shard.barrier()


def max_over_ranks(x):
    if not _DIST["on"]:
        return x
    from paper_2607_19456_b200 import shard
    return shard.reduce_step_time(x, device=_DIST["device"])


# --------------------------------------------------------------------------------------
# starting the ranks (plain `python bench.py --gpus N`)
# --------------------------------------------------------------------------------------
def free_port():
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def rank_env(rank, world, port, base=None):
    """Environment of one child rank: what torchrun would have set, rendezvous on 127.0.0.1."""
    env = dict(os.environ if base is None else base)
    env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
               MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    return env


def spawn_ranks(world, argv):
    """One child process per GPU running this script with the same arguments; rank 0 prints
    the JSON line.  Returns the first non-zero exit code (children still running are then
    terminated by their PIDs)."""
    import subprocess
    port = free_port()
    procs = [subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=rank_env(r, world, port))
             for r in range(world)]
    rc = 0
    pending = list(procs)
    while pending:
        for p in list(pending):
            code = p.poll()
            if code is None:
                continue
            pending.remove(p)
            if code != 0 and rc == 0:
                rc = code
                for other in pending:
                    other.terminate()
        time.sleep(0.05)
    return rc


# --------------------------------------------------------------------------------------
# the CPU oracle as baseline / reference arm
# --------------------------------------------------------------------------------------
def oracle_units(w, q, K, V, units):
    """The first `units` (batch, kv head) groups as an independent batch with h_kv = 1."""
    g = w.group
    U = w.batch * w.h_kv
    qq = np.asarray(q).reshape(U, g, w.d_k)[:units]
    KK = np.asarray(K).reshape(U, 1, w.n, w.d_k)[:units]
    VV = np.asarray(V).reshape(U, 1, w.n, w.d_v)[:units]
    return qq, KK, VV


def time_oracle_sample(w, q, K, V, budget_s):
    """Time the oracle on a sample sized for about `budget_s` seconds.
    -> (seconds, units in the sample, sample bytes, oracle output for the sample)."""
    import oracle
    U = w.batch * w.h_kv
    qq, KK, VV = oracle_units(w, q, K, V, 1)
    t = time.perf_counter(); oracle.decode(qq, KK, VV, w.scale); t1 = time.perf_counter() - t
    thr = max(1, oracle.threads())
    per_unit_parallel = t1 * min(w.group, thr) / thr      # one unit alone keeps only g_s threads busy
    units = int(max(1, min(U, budget_s / max(per_unit_parallel, 1e-6))))
    qq, KK, VV = oracle_units(w, q, K, V, units)
    t = time.perf_counter(); out = oracle.decode(qq, KK, VV, w.scale); secs = time.perf_counter() - t
    nbytes = units * (w.n * (w.d_k + w.d_v) + w.group * (w.d_k + w.d_v)) * 4
    return secs, units, nbytes, out


def run_reference(args, wname):
    rank = env_int("RANK", 0)
    if rank != 0:
        return
    import oracle
    w = mi.WORKLOADS[wname] if wname in mi.WORKLOADS else EXTRA_WORKLOADS[wname]
    if wname == "multi_step":
        w = mi.small_like(w, n=int(np.mean([w.len_lo, w.len_hi])) + w.steps // 2)
    total = args.steps + args.warmup
    budget = max(0.05, min(2.0, 150.0 / max(1, total)))
    # only as much of the input as the sample can use is generated
    U = w.batch * w.h_kv
    probe = mi.small_like(w, batch=1, h_q=w.group, h_kv=1)
    secs, _, _, _ = time_oracle_sample(probe, probe.q(), probe.K(), probe.V(), 0.0)
    thr = max(1, oracle.threads())
    units = int(max(1, min(U, budget / max(secs * min(w.group, thr) / thr, 1e-6))))
    ws = mi.small_like(w, batch=units, h_q=w.group, h_kv=1)
    q, K, V = ws.q(), ws.K(), ws.V()
    nbytes = units * (w.n * (w.d_k + w.d_v) + w.group * (w.d_k + w.d_v)) * 4
    for _ in range(args.warmup):
        oracle.decode(q, K, V, w.scale)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.decode(q, K, V, w.scale)
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    gbs = nbytes / dt / 1e9
    sample = "%d of %d (batch, kv-head) groups per step, n=%d, g_s=%d" % (units, U, w.n, w.group)
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": wname, "sample": sample},
            "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": sample},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------
# one sampled parity figure per workload (oracle on one unit of the buffers just timed)
# --------------------------------------------------------------------------------------
def sampled_parity(run, w):
    """Max abs error of the last timed step's output against the oracle on a sample: for the
    dense workloads the first and the last (batch, kv head) unit of buffer set 0, for the
    multi-step workload sequence 0 (all heads).  The inputs are read back from the device."""
    import oracle
    if isinstance(run, MultiStepRun):
        if run.t == 0:
            return None
        lens = (run.lens0_h[:1] + run.t).astype(np.int32)
        q = run.q[run.t - 1, :1].cpu().numpy()
        ref = oracle.decode_varlen(q, run.K[:1].cpu().numpy(), run.V[:1].cpu().numpy(), lens, w.scale)
        return float(np.max(np.abs(run.out[:1].cpu().numpy().astype(np.float64) - ref)))
    used = (run.i - 1) % run.nsets if run.i > 0 else 0
    g, worst = w.group, 0.0
    for b, h in {(0, 0), (w.batch - 1, w.h_kv - 1)}:
        q = run.q[used, b:b + 1, h * g:(h + 1) * g].cpu().numpy()
        K = run.K[used, b:b + 1, h:h + 1].cpu().numpy()
        V = run.V[used, b:b + 1, h:h + 1].cpu().numpy()
        got = run.out[used, b:b + 1, h * g:(h + 1) * g].cpu().numpy()
        worst = max(worst, float(np.max(np.abs(got.astype(np.float64) - oracle.decode(q, K, V, w.scale)))))
    return worst


# --------------------------------------------------------------------------------------
# sequence split over the ranks (--split seq): one all-gather of partial triples per step
# --------------------------------------------------------------------------------------
class SeqSplitRun:
    """Every rank holds a contiguous range of the cached rows of every (batch, kv head) of one
    workload; a step is moa_decode_attn_partial over the local rows, one all-gather of
    batch * h_q * (d_v + 4) floats, and moa_combine_partials (in rank order)."""

    def __init__(self, w, rank, world, device="cuda"):
        import torch
        import paper_2607_19456_b200 as moa
        from paper_2607_19456_b200 import shard
        self.moa, self.torch, self.w, self.shard = moa, torch, w, shard
        start, count = shard.shard_rows(w.n, world, rank, align=128)
        self.n_local = count
        B, hq, hkv, dk, dv = w.batch, w.h_q, w.h_kv, w.d_k, w.d_v
        g = torch.Generator(device=device).manual_seed(w.seed + 17 * rank)
        self.nsets = 2
        self.q = torch.randn((B, hq, dk), device=device, generator=torch.Generator(device=device).manual_seed(w.seed))
        self.K = torch.randn((2, B, hkv, max(count, 1), dk), device=device, generator=g)
        self.V = torch.randn((2, B, hkv, max(count, 1), dv), device=device, generator=g)
        if w.v_dist == "uniform":
            self.V.uniform_(-1, 1, generator=g)
        self.out = torch.zeros((B, hq, dv), device=device)
        self.decode_bytes = moa.moa_min_bytes(B, hq, hkv, w.n, dk, dv)
        self.bytes_per_step = self.decode_bytes            # whole job (the rows of all ranks)
        self.i = 0
        self.l2_note = "rotating over 2 buffer sets of the local rows"

    def step(self):
        s = self.i % 2
        self.i += 1
        K = self.K[s][:, :, :self.n_local]
        V = self.V[s][:, :, :self.n_local]
        self.shard.seq_split_decode(self.q, K, V, self.out, self.w.scale)

    def reset(self):
        self.i = 0

    def profile(self, mode):
        self.moa.moa_profile(mode)

    def profile_read(self):
        return self.moa.moa_profile_read()


# --------------------------------------------------------------------------------------
def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(mi.WORKLOADS) + list(EXTRA_WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--split", default="batch", choices=["batch", "seq"],
                    help="what is cut over the ranks: the batch (no collective) or the cached rows (one all-gather)")
    ap.add_argument("--no-others", action="store_true", help="skip the timing-only lines of the other workloads")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling on a small case)")
    ap.add_argument("--n", type=int, default=0, help="override the workload's cached tokens (profiling on a small case)")
    args = ap.parse_args(argv)
    if args.warmup < 3:
        args.warmup = 3
    return args


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    args = parse_args(argv)
    if args.impl == "reference":
        run_reference(args, args.workload)
        return 0
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args.gpus, argv)               # the children come back here with the rank environment
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libmoa has no CPU path")
    run_rank(args, CudaSide(env_int("LOCAL_RANK", 0)))
    return 0


def run_rank(args, side, make_run=None):
    """One rank of the benchmark.  `make_run(workload, rank, world)` (tests only) replaces the
    object whose step() is timed."""
    import torch
    rank, world, local = env_int("RANK", 0), env_int("WORLD_SIZE", 1), env_int("LOCAL_RANK", 0)
    wname = args.workload
    on_gpu = isinstance(side, CudaSide)
    if world > 1:
        import torch.distributed as dist
        if on_gpu:
            dist.init_process_group(side.backend, device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(side.backend)
        _DIST["on"], _DIST["device"] = True, side.device
    moa = None
    if on_gpu:
        import paper_2607_19456_b200 as moa
        moa.lib()                                       # fail loudly if the library is missing

    w = mi.WORKLOADS[wname] if wname in mi.WORKLOADS else EXTRA_WORKLOADS[wname]
    if args.batch > 0:
        w = mi.small_like(w, batch=args.batch)
    if args.n > 0 and wname != "multi_step":
        w = mi.small_like(w, n=args.n)
    seq_split = args.split == "seq" and wname != "multi_step"
    if make_run is not None:
        run = make_run(w, rank, world)
    elif seq_split:
        run = SeqSplitRun(w, rank, world)
    elif wname == "multi_step":
        args.steps = min(args.steps, w.steps - args.warmup)
        run = MultiStepRun(w, seed_shift=rank)
    else:
        run = DenseRun(w, seed_shift=rank, host_inputs=True)

    l2_note = run.l2_note
    sampler = ClockSampler(local) if on_gpu else None
    ms, _, launches, clocks, segs = time_steps(run, args.steps, args.warmup, side, sampler, segment=min(300, args.steps // 2))
    per_rank = ms
    ms = max_over_ranks(ms)
    per_rank_all = None
    if world > 1:
        import torch.distributed as dist
        per_rank_all = [None] * world
        dist.all_gather_object(per_rank_all, per_rank * 1e3)
    # second pass: the same steps with an event pair around every launch of the dominant kernel
    kern_ms = None
    if on_gpu:
        _, kern_ms, _, _, _ = time_steps(run, min(args.steps, 200), 3, side, None, bracket=True)
    if wname == "multi_step" and make_run is None:
        step_bytes = run.bytes_for_steps(0, args.steps) / args.steps
        decode_bytes = step_bytes
    else:
        step_bytes, decode_bytes = run.bytes_per_step, run.decode_bytes
    ranks_of_work = 1 if seq_split else world             # seq split: the bytes already are the whole job's
    value = ranks_of_work * step_bytes / (ms * 1e-3) / 1e9

    peak, peak_kind = measured_hbm_peak()
    roof = None
    single_launch = (launches == args.steps)
    if on_gpu and (single_launch or kern_ms):
        # One launch per step: the kernel's average launch duration over the timed region is
        # the event-timed region divided by its launches (this includes the gap between
        # launches, and no per-launch event overhead).  Otherwise: the bracketed figure.
        k_ms = ms if single_launch else kern_ms
        kbytes = decode_bytes / (world if seq_split else 1)
        ach = kbytes / (k_ms * 1e-3) / 1e9
        kname = {moa.PATH_GENERIC: "generic_decode_kernel",
                 moa.PATH_STREAM: "stream_decode_kernel (FMA; scores, online softmax, weighted sum, append, partial merge)",
                 moa.PATH_GROUPED: "grouped64_decode_kernel (tcgen05; scores, online softmax, weighted sum)",
                 moa.PATH_MMA: "mma_decode_kernel (warp-level TF32 MMA; scores, online softmax, weighted sum, append, "
                               "partial merge)"}.get(moa.moa_last_path(), "?")
        roof = {"bound": "hbm", "kernel": kname, "achieved": ach, "peak": peak,
                "peak_source": "of " + peak_kind, "unit": "GB/s", "frac": ach / peak,
                "frac_of_nominal_8000": ach / 8000.0,
                "kernel_us_per_launch": k_ms * 1e3,
                "how": ("CUDA events around the %d back-to-back launches of the timed region / launches" % launches)
                if single_launch else "CUDA event pair around every launch of the kernel (second pass)",
                "kernel_us_per_launch_event_bracketed": (kern_ms * 1e3 if kern_ms else None),
                "kernel_us_event_bracketed_min_median_max": (
                    [min(LAST_BRACKETED), statistics.median(LAST_BRACKETED), max(LAST_BRACKETED)] if LAST_BRACKETED else None),
                "algorithmic_bytes_per_launch": kbytes,
                "traffic": ncu_traffic(wname)}
        if roof["traffic"] is not None and wname == "multi_step" and make_run is None:
            # captured on the loop's first step (the shortest caches); DRAM traffic grows in
            # proportion to the rows a step streams, so scale it to the timed region's mean step
            captured = run.bytes_for_steps(0, 1)
            roof["traffic"] = roof["traffic"] * kbytes / captured
            roof["traffic_how"] = ("ncu capture of step 0 (%d B for %d algorithmic bytes), scaled to the mean step"
                                   % (NCU_TRAFFIC[wname]["bytes"], captured))

    # ---- end to end through the host-buffer entry point --------------------------------
    e2e = None
    dense = isinstance(run, DenseRun)
    if dense and run.host is not None and args.e2e_steps > 0:
        run.e2e_step()                                   # warm-up: staging buffers are allocated here
        side.sync()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            run.e2e_step()
        dt = max_over_ranks((time.perf_counter() - t0) / args.e2e_steps)
        hb, db = run.e2e_bytes()
        e2e = {"value": world * run.decode_bytes / dt / 1e9, "unit": UNIT, "ms_per_step": dt * 1e3,
               "steps": args.e2e_steps, "h2d_bytes_per_step": hb, "d2h_bytes_per_step": db,
               "api": "moa_decode_attn_host (pinned host q,K,V,out; copies inside the timed region)"}
        # the same step with the cache resident on the device (what a decode loop does): only the
        # token's q, k, v travel host -> device and the output device -> host, every step
        n_res = max(20, args.e2e_steps)
        run.resident_step()
        t0 = time.perf_counter()
        for _ in range(n_res):
            run.resident_step()
        dtr = max_over_ranks((time.perf_counter() - t0) / n_res)
        e2e["resident_cache"] = {
            "value": world * run.bytes_per_step / dtr / 1e9, "unit": UNIT, "ms_per_step": dtr * 1e3, "steps": n_res,
            "h2d_bytes_per_step": (w.batch * w.h_q * w.d_k + w.batch * w.h_kv * (w.d_k + w.d_v)) * 4,
            "d2h_bytes_per_step": w.batch * w.h_q * w.d_v * 4,
            "api": "pinned q, k_new, v_new -> device; moa_append_decode; out -> pinned host; synchronised every step"}
    elif wname == "multi_step":
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
               "note": "the multi-step cache lives on the device by definition; no host-buffer variant"}

    # ---- CPU oracle beside it (rank 0, N = 1 only) -------------------------------------
    cpu = None
    parity = None
    if rank == 0 and world == 1 and on_gpu and not args.no_cpu:
        parity = sampled_parity(run, w)
    if rank == 0 and world == 1 and dense and not args.no_cpu:
        import oracle
        h = run.host
        Kh, Vh = h["K"].numpy(), h["V"].numpy()
        pos = np.full((w.batch,), w.n - 1, np.int32)
        oracle.kv_append(Kh, Vh, run.k_new_h, run.v_new_h, pos)     # what the timed steps did
        secs, units, nbytes, ref = time_oracle_sample(w, h["q"].numpy(), Kh, Vh, 15.0)
        # repeat the same sample until about 10 s of wall time have gone into the oracle
        passes, spent, best = 1, secs, secs
        qq, KK, VV = oracle_units(w, h["q"].numpy(), Kh, Vh, units)
        while spent < 10.0 and passes < 200:
            t0 = time.perf_counter(); oracle.decode(qq, KK, VV, w.scale); dt = time.perf_counter() - t0
            spent += dt; passes += 1; best = min(best, dt)
        secs = spent / passes
        used = (run.i - 1) % run.nsets if run.i > 0 else 0
        got = run.out[used].cpu().numpy().reshape(w.batch * w.h_kv, w.group, w.d_v)[:units]
        parity = max(parity or 0.0, float(np.max(np.abs(got.astype(np.float64) - ref.astype(np.float64)))))
        # the single-precision evaluation of the same definition, same sample, same cores
        f32_passes, f32_spent = 0, 0.0
        while f32_passes < 3 and f32_spent < 8.0:
            t0 = time.perf_counter(); oracle.decode_f32(qq, KK, VV, w.scale); f32_spent += time.perf_counter() - t0
            f32_passes += 1
        f32_secs = f32_spent / f32_passes
        cpu = {"value": nbytes / secs / 1e9, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
               "sample": "%d of %d (batch, kv-head) groups of the same inputs; mean of %d passes, %.1f s of wall time in total" %
                         (units, w.batch * w.h_kv, passes, spent),
               "us_per_step_extrapolated": secs * 1e6 * (w.batch * w.h_kv) / units,
               "best_pass_s": best,
               "single_precision_variant": {"value": nbytes / f32_secs / 1e9, "unit": UNIT, "passes": f32_passes,
                                            "us_per_step_extrapolated": f32_secs * 1e6 * (w.batch * w.h_kv) / units}}

    # ---- the other workloads (device-generated inputs): timing and one sampled parity each ----
    others = []
    if rank == 0 and world == 1 and on_gpu and not args.no_others and make_run is None:
        del run
        torch.cuda.empty_cache()
        for name, ow in list(mi.WORKLOADS.items()) + list(EXTRA_WORKLOADS.items()):
            if name == wname:
                continue
            try:
                if name == "multi_step":
                    r = MultiStepRun(ow)
                    k = min(200, ow.steps - 10)
                    oms, _, _, _, _ = time_steps(r, k, 10, side)
                    _, okern, _, _, _ = time_steps(r, k, 3, side, None, bracket=True)
                    ob = r.bytes_for_steps(0, k) / k
                    odec = ob
                else:
                    r = DenseRun(ow, host_inputs=False)
                    k = 600 if name == "mqa_long" else 100
                    oms, _, _, _, osegs = time_steps(r, k, 10, side, segment=200)
                    _, okern, _, _, _ = time_steps(r, 100, 3, side, None, bracket=True)
                    ob, odec = r.bytes_per_step, r.decode_bytes
                others.append({"workload": name, "us_per_step": oms * 1e3, "GBps": ob / (oms * 1e-3) / 1e9,
                               "frac_of_peak": ob / (oms * 1e-3) / 1e9 / peak,
                               "decode_kernel_us": okern * 1e3 if okern else None,
                               "decode_kernel_GBps": (odec / (okern * 1e-3) / 1e9) if okern else None,
                               "decode_kernel_frac_of_peak": (odec / (okern * 1e-3) / 1e9 / peak) if okern else None,
                               "frac_of_nominal_8000": ob / (oms * 1e-3) / 1e9 / 8000.0,
                               "decode_kernel_us_min_median_max": (
                                   [min(LAST_BRACKETED), statistics.median(LAST_BRACKETED), max(LAST_BRACKETED)]
                                   if LAST_BRACKETED else None),
                               "parity_max_abs_err_vs_oracle": (None if args.no_cpu else sampled_parity(r, ow)),
                               "l2": r.l2_note})
                if name != "multi_step" and osegs:
                    others[-1]["us_per_step_first_last_200"] = [osegs[0] * 1e3, osegs[1] * 1e3]
                if name == "single_head":              # latency-bound: also with its lines resident in L2
                    r.nsets = 1
                    wms, _, _, _, _ = time_steps(r, 200, 10, side)
                    others[-1]["us_per_step_l2_warm"] = wms * 1e3
                del r
                torch.cuda.empty_cache()
            except Exception as ex:                     # a secondary line must not lose the main one
                others.append({"workload": name, "error": repr(ex)[:200]})

    if rank == 0:
        if seq_split:
            step_desc = ("sequence split: moa_decode_attn_partial over %d local rows + all-gather of the partial triples "
                         "+ moa_combine_partials" % run.n_local)
            par = "sp%d (cached rows cut over the ranks, one all-gather per step)" % world
        else:
            step_desc = ("moa_decode_step: append + attend over ragged lengths + length advance, one launch" if wname == "multi_step"
                         else "moa_append_decode: kv append at row n-1 + decode attention over n rows, %d launch(es) per step"
                         % max(1, launches // max(1, args.steps)))
            par = "dp%d (batch-sharded, no collective)" % world
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "strong" if seq_split else "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": wname, "batch_per_gpu": w.batch, "h_q": w.h_q, "h_kv": w.h_kv,
                           "n": w.n, "d_k": w.d_k, "d_v": w.d_v, "parallelism": par, "step": step_desc, "l2": l2_note},
                "us_per_step": ms * 1e3, "us_per_step_per_rank": per_rank_all,
                "us_per_step_first_last_segment": ({"steps": min(300, args.steps // 2), "first": segs[0] * 1e3, "last": segs[1] * 1e3} if segs else None),
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
                "roofline": roof, "cpu_baseline": cpu, "parity_max_abs_err_vs_oracle": parity,
                "other_workloads": others}
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    sys.exit(main())

#!/usr/bin/env python
"""Benchmark of the decode-attention hot path (libmoa) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one pass of the whole hot path over one batch of synthetic input: the
KV-cache append of the new token's (k, v) row followed by decode attention over the
cache (for the multi-step workload: one fused append+attend step over ragged lengths).
Prints ONE JSON line (rank 0).  `value` is the achieved algorithmic HBM bandwidth of the
whole job (bytes of the paper's traffic model per step, summed over ranks, divided by
the step time, max over ranks); `ms_per_step` is the step time.

With N > 1 (launched under torchrun, one rank per GPU) every rank runs its own shard of
an N-times larger batch: the path has no exchange step, so there is no data-path
collective and the scaling is weak.

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
# (dram__bytes_read.sum + dram__bytes_write.sum), per workload; the summaries these come
# from are kept as text under profiles/.  None = not captured.
NCU_TRAFFIC_BYTES = {
    "gqa": 1074650112 + 3750144,        # profiles/stream_decode_kernel_gqa.md (full-size launch)
    "mqa_long": 537066496 + 314112,     # profiles/grouped64_decode_kernel_mqa_long.md (full-size launch)
    "extra_group8_d128": 1075588864 + 4157440,   # profiles/mma_decode_kernel_group8_d128.md (full-size launch)
}


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
}


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
        self.nsets = 1 if one >= 2 * L2_BYTES_ASSUMED else min(4096, -(-2 * L2_BYTES_ASSUMED // one))
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
        self.l2_note = ("inputs larger than L2 (%.0f MB per step)" % (one / 1e6)) if S == 1 else \
            ("rotating over %d buffer sets (%.0f MB total, larger than L2)" % (S, S * one / 1e6))

    def step(self):
        w, m = self.w, self.moa
        q, K, V, out = self.ptrs[self.i % self.nsets]
        kn, vn, pos = self.aux
        self.i += 1
        m.moa_append_decode(q, K, V, kn, vn, out, pos, w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale,
                            self.wsptr, self.ws_bytes, self.stream)

    def reset(self):
        self.i = 0
        # every sequence of this workload has n rows after the append: tell the library (it cannot
        # see the lengths, which live on the device)
        self.moa.moa_set_option(self.moa.OPT_MIN_ROWS_HINT, self.w.n)

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
        self.moa.moa_set_option(self.moa.OPT_MIN_ROWS_HINT, 0)     # ragged lengths from 512 rows: no promise


def time_steps(run, steps, warmup, sampler=None, bracket=False):
    """-> (ms per step, decode-kernel ms per launch or None, launches in the timed region, clocks).
    With bracket=True the library also records a CUDA event pair around every launch of
    the dominant decode kernel (which costs a few microseconds per launch)."""
    import torch
    moa = run.moa
    run.reset()
    for _ in range(warmup):
        run.step()
    torch.cuda.synchronize()
    if isinstance(run, MultiStepRun):
        run.reset()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    moa.moa_profile(2 if bracket else 1)
    e0.record()
    for _ in range(steps):
        run.step()
    e1.record()
    torch.cuda.synchronize()
    kern_ms, kern_n, launches = moa.moa_profile_read()
    LAST_BRACKETED.clear()
    if bracket and kern_n:
        LAST_BRACKETED.extend(moa.moa_profile_launch_ms(i) * 1e3 for i in range(int(kern_n)))
    moa.moa_profile(0)
    clocks = sampler.stop() if sampler else None
    barrier()
    ms = e0.elapsed_time(e1) / steps
    return ms, (kern_ms / kern_n if kern_n else None), launches, clocks


_DIST = {"on": False}
LAST_BRACKETED = []      # per-launch event times (us) of the last bracketed pass


def barrier():
    if _DIST["on"]:
        from paper_2607_19456_b200 import shard
        shard.barrier()


def max_over_ranks(x):
    if not _DIST["on"]:
        return x
    from paper_2607_19456_b200 import shard
    return shard.reduce_step_time(x, device="cuda")


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
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(mi.WORKLOADS) + list(EXTRA_WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-others", action="store_true", help="skip the timing-only lines of the other workloads")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling on a small case)")
    ap.add_argument("--n", type=int, default=0, help="override the workload's cached tokens (profiling on a small case)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    wname = args.workload

    if args.impl == "reference":
        run_reference(args, wname)
        return

    import torch
    import paper_2607_19456_b200 as moa

    rank, world, local = env_int("RANK", 0), env_int("WORLD_SIZE", 1), env_int("LOCAL_RANK", 0)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libmoa has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        _DIST["on"] = True
    moa.lib()                                           # fail loudly if the library is missing

    w = mi.WORKLOADS[wname] if wname in mi.WORKLOADS else EXTRA_WORKLOADS[wname]
    if args.batch > 0:
        w = mi.small_like(w, batch=args.batch)
    if args.n > 0 and wname != "multi_step":
        w = mi.small_like(w, n=args.n)
    if wname == "multi_step":
        args.steps = min(args.steps, w.steps - args.warmup)
        run = MultiStepRun(w, seed_shift=rank)
    else:
        run = DenseRun(w, seed_shift=rank, host_inputs=True)

    l2_note = run.l2_note
    sampler = ClockSampler(local)
    ms, _, launches, clocks = time_steps(run, args.steps, args.warmup, sampler)
    ms = max_over_ranks(ms)
    # second pass: the same steps with an event pair around every launch of the dominant kernel
    bsteps = min(args.steps, 200)
    _, kern_ms, _, _ = time_steps(run, bsteps, 3, None, bracket=True)
    if wname == "multi_step":
        step_bytes = run.bytes_for_steps(0, args.steps) / args.steps
        decode_bytes = step_bytes
    else:
        step_bytes, decode_bytes = run.bytes_per_step, run.decode_bytes
    value = world * step_bytes / (ms * 1e-3) / 1e9

    peak, peak_kind = measured_hbm_peak()
    roof = None
    single_launch = (launches == args.steps)
    if single_launch or kern_ms:
        # One launch per step: the kernel's average launch duration over the timed region is
        # the event-timed region divided by its launches (this includes the gap between
        # launches, and no per-launch event overhead).  Otherwise: the bracketed figure.
        k_ms = ms if single_launch else kern_ms
        ach = decode_bytes / (k_ms * 1e-3) / 1e9
        kname = {moa.PATH_GENERIC: "generic_decode_kernel",
                 moa.PATH_STREAM: "stream_decode_kernel (FMA; scores, online softmax, weighted sum, append, partial merge)",
                 moa.PATH_GROUPED: "grouped64_decode_kernel / grouped_decode_kernel (tcgen05)",
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
                "algorithmic_bytes_per_launch": decode_bytes,
                "traffic": NCU_TRAFFIC_BYTES.get(wname)}

    # ---- end to end through the host-buffer entry point --------------------------------
    e2e = None
    if wname != "multi_step" and run.host is not None and args.e2e_steps > 0:
        run.e2e_step()                                   # warm-up: staging buffers are allocated here
        torch.cuda.synchronize()
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
    if rank == 0 and world == 1 and not args.no_cpu and wname != "multi_step":
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
        got = run.out[0].cpu().numpy().reshape(w.batch * w.h_kv, w.group, w.d_v)[:units]
        parity = float(np.max(np.abs(got.astype(np.float64) - ref.astype(np.float64))))
        cpu = {"value": nbytes / secs / 1e9, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
               "sample": "%d of %d (batch, kv-head) groups of the same inputs; mean of %d passes, %.1f s of wall time in total" %
                         (units, w.batch * w.h_kv, passes, spent),
               "us_per_step_extrapolated": secs * 1e6 * (w.batch * w.h_kv) / units,
               "best_pass_s": best}

    # ---- the other workloads, timing only (device-generated inputs) ---------------------
    others = []
    if rank == 0 and world == 1 and not args.no_others:
        del run
        torch.cuda.empty_cache()
        for name, ow in list(mi.WORKLOADS.items()) + list(EXTRA_WORKLOADS.items()):
            if name == wname:
                continue
            try:
                if name == "multi_step":
                    r = MultiStepRun(ow)
                    k = min(200, ow.steps - 10)
                    oms, _, _, _ = time_steps(r, k, 10)
                    _, okern, _, _ = time_steps(r, k, 3, None, bracket=True)
                    ob = r.bytes_for_steps(0, k) / k
                    odec = ob
                else:
                    r = DenseRun(ow, host_inputs=False)
                    oms, _, _, _ = time_steps(r, 100, 10)
                    _, okern, _, _ = time_steps(r, 100, 3, None, bracket=True)
                    ob, odec = r.bytes_per_step, r.decode_bytes
                others.append({"workload": name, "us_per_step": oms * 1e3, "GBps": ob / (oms * 1e-3) / 1e9,
                               "decode_kernel_us": okern * 1e3 if okern else None,
                               "decode_kernel_GBps": (odec / (okern * 1e-3) / 1e9) if okern else None,
                               "decode_kernel_frac_of_peak": (odec / (okern * 1e-3) / 1e9 / peak) if okern else None,
                               "frac_of_nominal_8000": ob / (oms * 1e-3) / 1e9 / 8000.0,
                               "decode_kernel_us_min_median_max": (
                                   [min(LAST_BRACKETED), statistics.median(LAST_BRACKETED), max(LAST_BRACKETED)]
                                   if LAST_BRACKETED else None),
                               "l2": r.l2_note})
                if name == "single_head":              # latency-bound: also with its lines resident in L2
                    r.nsets = 1
                    wms, _, _, _ = time_steps(r, 200, 10)
                    others[-1]["us_per_step_l2_warm"] = wms * 1e3
                del r
                torch.cuda.empty_cache()
            except Exception as ex:                     # a secondary line must not lose the main one
                others.append({"workload": name, "error": repr(ex)[:200]})

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": wname, "batch_per_gpu": w.batch, "h_q": w.h_q, "h_kv": w.h_kv,
                           "n": w.n, "d_k": w.d_k, "d_v": w.d_v, "parallelism": "dp%d (batch-sharded, no collective)" % world,
                           "step": ("moa_decode_step: append + attend over ragged lengths + length advance, one launch" if wname == "multi_step"
                                    else "moa_append_decode: kv append at row n-1 + decode attention over n rows (MOA_OPT_MIN_ROWS_HINT = n), %d launch(es) per step"
                                    % max(1, launches // max(1, args.steps))),
                           "l2": l2_note},
                "us_per_step": ms * 1e3, "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
                "roofline": roof, "cpu_baseline": cpu, "parity_max_abs_err_vs_oracle": parity,
                "other_workloads": others}
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

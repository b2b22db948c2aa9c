"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA library's tests.

This module holds none of the method's arithmetic: only a counter-based random
generator and the table of workload shapes.  Every element of a tensor is a pure
function of (seed, tensor id, flat element index), so

* results do not depend on thread count or chunking,
* any sub-range of a tensor (for example one K/V slab of a 1 GiB cache) can be
  regenerated on its own, which is how full-size runs are spot-checked against the
  oracle without the oracle ever touching the whole tensor.

Generator: a 64-bit mix (the splitmix64 finaliser) of the counter gives a uniform in
(0,1); normals come from Box-Muller in double precision on the pair
(element 2p, element 2p+1) and are rounded once to fp32.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GOLD = 0x9E3779B97F4A7C15
_MASK = (1 << 64) - 1

# tensor ids
TID_Q, TID_K, TID_V, TID_KNEW, TID_VNEW, TID_LENS, TID_QSTEP = 1, 2, 3, 4, 5, 6, 7

_CHUNK = 1 << 21
_POOL = None


def _pool():
    global _POOL
    if _POOL is None:
        _POOL = ThreadPoolExecutor(max_workers=max(1, min(32, os.cpu_count() or 1)))
    return _POOL


def _key(seed: int, tid: int) -> np.uint64:
    return np.uint64((seed * _GOLD + tid * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & _MASK)


def _mix(counter: np.ndarray, key: np.uint64) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = counter + key
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def _u01(counter: np.ndarray, key: np.uint64) -> np.ndarray:
    """Uniform in the open interval (0, 1), 53 bits."""
    z = _mix(counter, key)
    return ((z >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _normal_range(key: np.uint64, start: int, stop: int) -> np.ndarray:
    p0, p1 = start // 2, (stop + 1) // 2
    p = np.arange(p0, p1, dtype=np.uint64)
    u1 = _u01(p * np.uint64(2), key)
    u2 = _u01(p * np.uint64(2) + np.uint64(1), key)
    r = np.sqrt(-2.0 * np.log(u1))
    th = (2.0 * np.pi) * u2
    z = np.empty(2 * (p1 - p0), np.float64)
    z[0::2] = r * np.cos(th)
    z[1::2] = r * np.sin(th)
    return z[start - 2 * p0: stop - 2 * p0].astype(np.float32)


def _uniform_range(key: np.uint64, start: int, stop: int) -> np.ndarray:
    i = np.arange(start, stop, dtype=np.uint64)
    return (2.0 * _u01(i, key) - 1.0).astype(np.float32)


def _fill(fn, key, start, stop, out=None):
    n = stop - start
    if out is None:
        out = np.empty(n, np.float32)
    if n <= _CHUNK:
        out[:n] = fn(key, start, stop)
        return out
    bounds = list(range(start, stop, _CHUNK)) + [stop]

    def work(k):
        a, b = bounds[k], bounds[k + 1]
        out[a - start: b - start] = fn(key, a, b)

    list(_pool().map(work, range(len(bounds) - 1)))
    return out


def normal(seed: int, tid: int, shape, start: int = 0, out=None) -> np.ndarray:
    """iid N(0,1) fp32 tensor of ``shape``; element i is element ``start + i`` of the
    (seed, tid) stream.  ``out`` (flat fp32, e.g. a view of pinned memory) is filled in
    place when given."""
    n = int(np.prod(shape))
    flat = _fill(_normal_range, _key(seed, tid), start, start + n,
                 None if out is None else out.reshape(-1))
    return flat.reshape(shape)


def uniform(seed: int, tid: int, shape, start: int = 0, out=None) -> np.ndarray:
    """iid U(-1,1) fp32 tensor of ``shape`` (same addressing as :func:`normal`)."""
    n = int(np.prod(shape))
    flat = _fill(_uniform_range, _key(seed, tid), start, start + n,
                 None if out is None else out.reshape(-1))
    return flat.reshape(shape)


def integers(seed: int, tid: int, count: int, lo: int, hi: int) -> np.ndarray:
    """``count`` iid integers uniform in [lo, hi] (inclusive), int32."""
    u = _u01(np.arange(count, dtype=np.uint64), _key(seed, tid))
    return (lo + np.floor(u * (hi - lo + 1)).astype(np.int64)).clip(lo, hi).astype(np.int32)


@dataclass(frozen=True)
class Workload:
    """One synthetic decode workload.  ``v_dist`` is 'normal' or 'uniform'."""
    name: str
    seed: int
    batch: int
    h_q: int
    h_kv: int
    n: int            # cached tokens (dense workloads) / row capacity (multi-step)
    d_k: int
    d_v: int
    v_dist: str = "normal"
    # multi-step only
    steps: int = 0
    len_lo: int = 0
    len_hi: int = 0

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(np.float64(self.d_k)))

    @property
    def group(self) -> int:
        return self.h_q // self.h_kv

    def q(self, out=None):
        return normal(self.seed, TID_Q, (self.batch, self.h_q, self.d_k), out=out)

    def K(self, out=None):
        return normal(self.seed, TID_K, (self.batch, self.h_kv, self.n, self.d_k), out=out)

    def V(self, out=None):
        fn = normal if self.v_dist == "normal" else uniform
        return fn(self.seed, TID_V, (self.batch, self.h_kv, self.n, self.d_v), out=out)

    def K_slab(self, b: int, h: int, rows: int | None = None):
        """Rows [0, rows) of K[b, h] regenerated on their own."""
        rows = self.n if rows is None else rows
        off = ((b * self.h_kv + h) * self.n) * self.d_k
        return normal(self.seed, TID_K, (rows, self.d_k), start=off)

    def V_slab(self, b: int, h: int, rows: int | None = None):
        rows = self.n if rows is None else rows
        off = ((b * self.h_kv + h) * self.n) * self.d_v
        fn = normal if self.v_dist == "normal" else uniform
        return fn(self.seed, TID_V, (rows, self.d_v), start=off)

    # ---- multi-step (cache capacity n, ragged start lengths) -------------------
    def start_lens(self) -> np.ndarray:
        return integers(self.seed, TID_LENS, self.batch, self.len_lo, self.len_hi)

    def k_new(self, step: int):
        per = self.batch * self.h_kv * self.d_k
        return normal(self.seed, TID_KNEW, (self.batch, self.h_kv, self.d_k), start=step * per)

    def v_new(self, step: int):
        per = self.batch * self.h_kv * self.d_v
        return normal(self.seed, TID_VNEW, (self.batch, self.h_kv, self.d_v), start=step * per)

    def q_step(self, step: int):
        per = self.batch * self.h_q * self.d_k
        return normal(self.seed, TID_QSTEP, (self.batch, self.h_q, self.d_k), start=step * per)


# The five benchmark workloads (shapes and distributions as the benchmark definition
# states them; seeds 1001..1005).
WORKLOADS = {
    "single_head": Workload("single_head", 1001, 1, 1, 1, 256, 64, 64),
    "mha": Workload("mha", 1002, 8, 32, 32, 4096, 128, 128),
    "gqa": Workload("gqa", 1003, 16, 32, 8, 8192, 128, 128),
    "mqa_long": Workload("mqa_long", 1004, 4, 64, 1, 131072, 128, 128, v_dist="uniform"),
    "multi_step": Workload("multi_step", 1005, 32, 32, 8, 2560, 128, 128,
                           steps=512, len_lo=512, len_hi=2048),
}


def small_like(w: Workload, **kw) -> Workload:
    """A reduced copy of a workload (same structure, smaller sizes) for quick parity."""
    from dataclasses import replace
    return replace(w, **kw)


# ---------------------------------------------------------------------------------------
# Low-entropy attention: inputs whose softmax mass sits on a few rows, so that no error
# averages out over the cache.  Pure input shaping (no arithmetic of the method): the query
# heads of a group share a common direction c, and a cached key is placed at a chosen score
# level t by making it (t * sqrt(d) / |c|^2) * c plus a little noise.
# ---------------------------------------------------------------------------------------
TID_COMMON, TID_QNOISE, TID_KNOISE = 11, 12, 13


def _group_common(seed, B, h_kv, d):
    return normal(seed, TID_COMMON, (B, h_kv, d)).astype(np.float64)


def peaked_case(seed, B, h_q, h_kv, n, d, peaks, floor=12.0, v_gap=3.0, q_spread=0.3, d_v=None):
    """q, K, V (fp32) of a dense cache in which the rows listed in ``peaks`` = [(row, level), ...]
    score about ``level`` (natural units, after the 1/sqrt(d) scale) for every query head and all
    other rows about ``-floor`` + N(0, ~1).  The V rows of the peaks alternate between about
    +v_gap and -v_gap.  Rows may be negative (counted from the end)."""
    d_v = d if d_v is None else d_v
    g_s = h_q // h_kv
    c = _group_common(seed, B, h_kv, d)                                  # [B, h_kv, d]
    c2 = np.sum(c * c, axis=-1, keepdims=True)
    unit = c * (np.sqrt(float(d)) / c2)                                  # scores 1.0 against q = c
    q = np.repeat(c, g_s, axis=1) + q_spread * normal(seed, TID_QNOISE, (B, h_q, d)).astype(np.float64)
    K = normal(seed, TID_K, (B, h_kv, n, d)).astype(np.float64) - floor * unit[:, :, None, :]
    V = normal(seed, TID_V, (B, h_kv, n, d_v)).astype(np.float64)
    kn = normal(seed, TID_KNOISE, (B, h_kv, len(peaks), d)).astype(np.float64)
    for i, (row, level) in enumerate(peaks):
        K[:, :, row, :] = level * unit + 0.1 * kn[:, :, i, :]
        V[:, :, row, :] += v_gap if i % 2 == 0 else -v_gap
    return q.astype(np.float32), K.astype(np.float32), V.astype(np.float32)


def sorted_case(seed, B, h_q, h_kv, n, d, lo=-10.0, hi=10.0, descending=False, q_spread=0.3):
    """q, K, V (fp32) whose scores run monotonically from ``lo`` to ``hi`` along the cache
    (or the other way round): every tile raises -- or never raises -- the running maximum."""
    g_s = h_q // h_kv
    c = _group_common(seed, B, h_kv, d)
    c2 = np.sum(c * c, axis=-1, keepdims=True)
    unit = c * (np.sqrt(float(d)) / c2)
    q = np.repeat(c, g_s, axis=1) + q_spread * normal(seed, TID_QNOISE, (B, h_q, d)).astype(np.float64)
    levels = np.linspace(hi, lo, n) if descending else np.linspace(lo, hi, n)
    K = levels[None, None, :, None] * unit[:, :, None, :] + 0.05 * normal(seed, TID_K, (B, h_kv, n, d)).astype(np.float64)
    V = normal(seed, TID_V, (B, h_kv, n, d)).astype(np.float64)
    return q.astype(np.float32), K.astype(np.float32), V.astype(np.float32)

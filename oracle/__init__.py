"""ctypes access to the plain-C CPU oracle (``moa_oracle.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline leg
may import this package; the CUDA library and its Python binding never do, and this
package never imports them.  All arrays are numpy, host memory, C-contiguous.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        fp, dp, ip = C.POINTER(C.c_float), C.POINTER(C.c_double), C.POINTER(C.c_int32)
        i, d = C.c_int, C.c_double
        L.moa_oracle_decode.argtypes = [fp, fp, fp, fp, i, i, i, i, i, i, d]
        L.moa_oracle_decode_varlen.argtypes = [fp, fp, fp, fp, i, i, i, ip, i, i, i, d]
        L.moa_oracle_decode_f64.argtypes = [dp, dp, dp, dp, i, i, i, i, i, i, d]
        L.moa_oracle_decode_f32.argtypes = [fp, fp, fp, fp, i, i, i, i, i, i, C.c_float]
        L.moa_oracle_kv_append.argtypes = [fp, fp, fp, fp, ip, i, i, i, i, i]
        L.moa_oracle_min_bytes.argtypes = [i, i, i, C.c_longlong, i, i]
        L.moa_oracle_min_bytes.restype = C.c_longlong
        L.moa_oracle_threads.restype = C.c_int
        _lib = L
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


def _shapes(q, K, V):
    batch, h_q, d_k = q.shape
    b2, h_kv, n, d_k2 = K.shape
    b3, h_kv2, n2, d_v = V.shape
    if not (batch == b2 == b3 and h_kv == h_kv2 and n == n2 and d_k == d_k2):
        raise ValueError("inconsistent q/K/V shapes")
    return batch, h_q, h_kv, n, d_k, d_v


def decode(q, K, V, scale):
    """q [B,h_q,d_k], K [B,h_kv,n,d_k], V [B,h_kv,n,d_v] (fp32) -> out [B,h_q,d_v] fp32.
    Algorithm 1 with double intermediates."""
    q, K, V = _c(q, np.float32), _c(K, np.float32), _c(V, np.float32)
    B, hq, hkv, n, dk, dv = _shapes(q, K, V)
    out = np.empty((B, hq, dv), np.float32)
    rc = lib().moa_oracle_decode(_p(q, C.c_float), _p(K, C.c_float), _p(V, C.c_float),
                                 _p(out, C.c_float), B, hq, hkv, n, dk, dv, float(scale))
    if rc != 0:
        raise ValueError("moa_oracle_decode: invalid argument")
    return out


def decode_varlen(q, K, V, seq_lens, scale):
    """As :func:`decode`, attending over rows [0, seq_lens[b]) of a capacity-n_max cache."""
    q, K, V = _c(q, np.float32), _c(K, np.float32), _c(V, np.float32)
    lens = _c(seq_lens, np.int32)
    B, hq, hkv, n_max, dk, dv = _shapes(q, K, V)
    if lens.shape != (B,):
        raise ValueError("seq_lens must have shape [batch]")
    out = np.empty((B, hq, dv), np.float32)
    rc = lib().moa_oracle_decode_varlen(_p(q, C.c_float), _p(K, C.c_float),
                                        _p(V, C.c_float), _p(out, C.c_float), B, hq, hkv,
                                        _p(lens, C.c_int32), n_max, dk, dv, float(scale))
    if rc != 0:
        raise ValueError("moa_oracle_decode_varlen: invalid argument")
    return out


def decode_f64(q, K, V, scale):
    """All-double variant (inputs and outputs float64)."""
    q, K, V = _c(q, np.float64), _c(K, np.float64), _c(V, np.float64)
    B, hq, hkv, n, dk, dv = _shapes(q, K, V)
    out = np.empty((B, hq, dv), np.float64)
    rc = lib().moa_oracle_decode_f64(_p(q, C.c_double), _p(K, C.c_double),
                                     _p(V, C.c_double), _p(out, C.c_double),
                                     B, hq, hkv, n, dk, dv, float(scale))
    if rc != 0:
        raise ValueError("moa_oracle_decode_f64: invalid argument")
    return out


def decode_f32(q, K, V, scale):
    """Algorithm 1 with every intermediate in single precision (timing baseline / sanity band)."""
    q, K, V = _c(q, np.float32), _c(K, np.float32), _c(V, np.float32)
    B, hq, hkv, n, dk, dv = _shapes(q, K, V)
    out = np.empty((B, hq, dv), np.float32)
    rc = lib().moa_oracle_decode_f32(_p(q, C.c_float), _p(K, C.c_float), _p(V, C.c_float),
                                     _p(out, C.c_float), B, hq, hkv, n, dk, dv,
                                     float(scale))
    if rc != 0:
        raise ValueError("moa_oracle_decode_f32: invalid argument")
    return out


def kv_append(K, V, k_new, v_new, pos):
    """In-place append into K [B,h_kv,n_max,d_k], V [B,h_kv,n_max,d_v] (fp32,
    C-contiguous, writable) of k_new [B,h_kv,d_k], v_new [B,h_kv,d_v] at row pos[b]."""
    for a in (K, V):
        if a.dtype != np.float32 or not a.flags.c_contiguous or not a.flags.writeable:
            raise ValueError("K and V must be writable C-contiguous float32 arrays")
    k_new, v_new = _c(k_new, np.float32), _c(v_new, np.float32)
    pos = _c(pos, np.int32)
    B, hkv, n_max, dk = K.shape
    dv = V.shape[3]
    if k_new.shape != (B, hkv, dk) or v_new.shape != (B, hkv, dv) or pos.shape != (B,):
        raise ValueError("inconsistent append shapes")
    rc = lib().moa_oracle_kv_append(_p(K, C.c_float), _p(V, C.c_float),
                                    _p(k_new, C.c_float), _p(v_new, C.c_float),
                                    _p(pos, C.c_int32), B, hkv, n_max, dk, dv)
    if rc != 0:
        raise ValueError("moa_oracle_kv_append: invalid argument (pos out of range?)")


def min_bytes(batch, h_q, h_kv, n, d_k, d_v):
    """The paper's traffic model (Proposition 1 with the GQA factor), in bytes."""
    return int(lib().moa_oracle_min_bytes(batch, h_q, h_kv, n, d_k, d_v))


def threads():
    return int(lib().moa_oracle_threads())

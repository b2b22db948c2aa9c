"""B200-native decode attention over a KV cache (libmoa) -- thin Python binding.

The functions here have the names and argument order of the C ABI in ``include/moa.h``
and do argument marshalling only: every step of the computation runs in the CUDA kernels
of ``libmoa.so``.  Tensor arguments are ``torch`` CUDA tensors (used for device memory
and streams, nothing else) or raw integer device addresses.  There is no CPU fallback:
if the shared library is missing or fails to load, importing succeeds but every call
raises :class:`MoaError`.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmoa.so")

OK, ERR_INVALID, ERR_UNSUPPORTED, ERR_ALIGN, ERR_CAPACITY, ERR_WORKSPACE, ERR_CUDA = range(7)
STATUS_APPEND_RANGE, STATUS_SEQLEN_RANGE, STATUS_WAIT_TIMEOUT = 1, 2, 4
OPT_FORCE_PATH, OPT_NUM_CTAS, OPT_GROUPED_HEADS, OPT_DEPENDENT_LAUNCH, OPT_GROUPED_OPERANDS = 1, 2, 3, 4, 5
OPT_WAIT_LIMIT, OPT_TEST_SKIP_COPY = 7, 8
NOALLOC_SCRATCH_BYTES = 4 << 20
PATH_AUTO, PATH_GENERIC, PATH_STREAM, PATH_GROUPED, PATH_MMA = 0, 1, 2, 3, 4

_lib = None


class MoaError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__("%s failed: %s (code %d)" % (what, strerror(code), code))


def lib():
    """The loaded ``libmoa.so`` (loads it on first use; never builds it)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libmoa.so is missing: run `python -m paper_2607_19456_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        p, i, f, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
        L.moa_decode_attn.argtypes = [p, p, p, p, i, i, i, i, i, i, f, p]
        L.moa_decode_attn_noalloc.argtypes = [p, p, p, p, i, i, i, i, i, i, f, p]
        L.moa_decode_attn_varlen.argtypes = [p, p, p, p, i, i, i, p, i, i, i, f, p, sz, p]
        L.moa_decode_attn_partial.argtypes = [p, p, p, p, i, i, i, i, i, i, f, p]
        L.moa_combine_partials.argtypes = [p, i, p, i, i, i, p]
        L.moa_decode_attn_layers.argtypes = [p, p, p, p, i, i, i, i, i, i, i, f, p]
        L.moa_workspace_bytes.argtypes = [i, i, i, i, i, i]
        L.moa_workspace_bytes.restype = sz
        L.moa_kv_append.argtypes = [p, p, p, p, p, i, i, i, i, i, p]
        L.moa_lens_add.argtypes = [p, i, i, p]
        L.moa_decode_step.argtypes = [p, p, p, p, p, p, p, i, i, i, i, i, i, f, p, sz, p]
        L.moa_append_decode.argtypes = [p, p, p, p, p, p, p, i, i, i, i, i, i, f, p, sz, p]
        ll3 = C.POINTER(C.c_longlong)
        L.moa_decode_attn_strided.argtypes = [p, p, p, p, p, i, i, i, i, i, i, f, ll3, ll3, p, sz, p]
        L.moa_kv_append_strided.argtypes = [p, p, p, p, p, i, i, i, i, i, ll3, ll3, p]
        L.moa_decode_step_strided.argtypes = [p, p, p, p, p, p, p, i, i, i, i, i, i, f, ll3, ll3, p, sz, p]
        L.moa_decode_attn_host.argtypes = [p, p, p, p, i, i, i, i, i, i, f]
        L.moa_device_status.argtypes = [p, C.POINTER(C.c_int)]
        L.moa_min_bytes.argtypes = [i, i, i, C.c_longlong, i, i]
        L.moa_min_bytes.restype = C.c_longlong
        L.moa_strerror.argtypes = [i]
        L.moa_strerror.restype = C.c_char_p
        L.moa_set_option.argtypes = [i, i]
        L.moa_profile.argtypes = [i]
        L.moa_profile_read.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_longlong),
                                       C.POINTER(C.c_longlong)]
        L.moa_profile_launch_ms.argtypes = [C.c_longlong, C.POINTER(C.c_double)]
        _lib = L
    return _lib


def _ptr(x):
    """Device (or host) address of a tensor / array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError("expected a tensor, an array or an address")


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(code, what):
    if code != OK:
        raise MoaError(code, what)


def strerror(code: int) -> str:
    return lib().moa_strerror(int(code)).decode()


def moa_decode_attn(q, K, V, out, batch, h_q, h_kv, n, d_k, d_v, scale, stream=None):
    _check(lib().moa_decode_attn(_ptr(q), _ptr(K), _ptr(V), _ptr(out), batch, h_q, h_kv, n, d_k,
                                 d_v, scale, _stream(stream)), "moa_decode_attn")


def moa_decode_attn_noalloc(q, K, V, out, batch, h_q, h_kv, n, d_k, d_v, scale, stream=None):
    """Same as :func:`moa_decode_attn`, for callers that may not allocate device memory:
    scratch comes from a fixed array inside the library (see ``include/moa.h``)."""
    _check(lib().moa_decode_attn_noalloc(_ptr(q), _ptr(K), _ptr(V), _ptr(out), batch, h_q, h_kv, n,
                                         d_k, d_v, scale, _stream(stream)), "moa_decode_attn_noalloc")


def moa_decode_attn_varlen(q, K, V, out, batch, h_q, h_kv, seq_lens, n_max, d_k, d_v, scale,
                           workspace, workspace_bytes, stream=None):
    _check(lib().moa_decode_attn_varlen(_ptr(q), _ptr(K), _ptr(V), _ptr(out), batch, h_q, h_kv,
                                        _ptr(seq_lens), n_max, d_k, d_v, scale, _ptr(workspace),
                                        workspace_bytes, _stream(stream)),
           "moa_decode_attn_varlen")


def moa_decode_attn_partial(q, K, V, partial, batch, h_q, h_kv, n, d_k, d_v, scale, stream=None):
    """Unnormalised triples over this device's rows: partial [batch, h_q, d_v + 4]."""
    _check(lib().moa_decode_attn_partial(_ptr(q), _ptr(K), _ptr(V), _ptr(partial), batch, h_q, h_kv, n,
                                         d_k, d_v, scale, _stream(stream)), "moa_decode_attn_partial")


def moa_combine_partials(partials, nparts, out, batch, h_q, d_v, stream=None):
    """Merge [nparts, batch, h_q, d_v + 4] triples into out [batch, h_q, d_v]."""
    _check(lib().moa_combine_partials(_ptr(partials), nparts, _ptr(out), batch, h_q, d_v, _stream(stream)),
           "moa_combine_partials")


def moa_decode_attn_layers(q, K, V, out, batch, h_q, h_kv, n, d_k, d_v, scale, stream=None):
    """q, K, V, out: sequences (one entry per layer) of tensors / addresses of one shape."""
    layers = len(q)
    arr = [(C.c_void_p * layers)(*[_ptr(x) for x in seq]) for seq in (q, K, V, out)]
    _check(lib().moa_decode_attn_layers(arr[0], arr[1], arr[2], arr[3], layers, batch, h_q, h_kv, n, d_k, d_v,
                                        scale, _stream(stream)), "moa_decode_attn_layers")


def moa_workspace_bytes(batch, h_q, h_kv, n_max, d_k, d_v) -> int:
    return int(lib().moa_workspace_bytes(batch, h_q, h_kv, n_max, d_k, d_v))


def moa_kv_append(K, V, k_new, v_new, pos, batch, h_kv, n_max, d_k, d_v, stream=None):
    _check(lib().moa_kv_append(_ptr(K), _ptr(V), _ptr(k_new), _ptr(v_new), _ptr(pos), batch, h_kv,
                               n_max, d_k, d_v, _stream(stream)), "moa_kv_append")


def moa_lens_add(lens, batch, delta, stream=None):
    _check(lib().moa_lens_add(_ptr(lens), batch, delta, _stream(stream)), "moa_lens_add")


def moa_decode_step(q, K, V, k_new, v_new, out, lens, batch, h_q, h_kv, n_max, d_k, d_v, scale,
                    workspace, workspace_bytes, stream=None):
    _check(lib().moa_decode_step(_ptr(q), _ptr(K), _ptr(V), _ptr(k_new), _ptr(v_new), _ptr(out),
                                 _ptr(lens), batch, h_q, h_kv, n_max, d_k, d_v, scale,
                                 _ptr(workspace), workspace_bytes, _stream(stream)),
           "moa_decode_step")


def moa_append_decode(q, K, V, k_new, v_new, out, pos, batch, h_q, h_kv, n_max, d_k, d_v, scale,
                      workspace, workspace_bytes, stream=None):
    _check(lib().moa_append_decode(_ptr(q), _ptr(K), _ptr(V), _ptr(k_new), _ptr(v_new), _ptr(out),
                                   _ptr(pos), batch, h_q, h_kv, n_max, d_k, d_v, scale,
                                   _ptr(workspace), workspace_bytes, _stream(stream)),
           "moa_append_decode")


def _strides3(st):
    """(batch, head, row) element strides as a host array of three long long."""
    if len(st) != 3:
        raise ValueError("strides are (batch, kv head, row) element counts")
    return (C.c_longlong * 3)(*[int(x) for x in st])


def moa_decode_attn_strided(q, K, V, out, seq_lens, batch, h_q, h_kv, n_max, d_k, d_v, scale, k_strides,
                            v_strides, workspace=None, workspace_bytes=0, stream=None):
    """K, V: base addresses (tensors or ints) of caches whose element (b, h, i, t) sits at
    base + b*strides[0] + h*strides[1] + i*strides[2] + t; seq_lens may be None."""
    _check(lib().moa_decode_attn_strided(_ptr(q), _ptr(K), _ptr(V), _ptr(out), _ptr(seq_lens), batch, h_q,
                                         h_kv, n_max, d_k, d_v, scale, _strides3(k_strides),
                                         _strides3(v_strides), _ptr(workspace), workspace_bytes,
                                         _stream(stream)), "moa_decode_attn_strided")


def moa_kv_append_strided(K, V, k_new, v_new, pos, batch, h_kv, n_max, d_k, d_v, k_strides, v_strides,
                          stream=None):
    _check(lib().moa_kv_append_strided(_ptr(K), _ptr(V), _ptr(k_new), _ptr(v_new), _ptr(pos), batch, h_kv,
                                       n_max, d_k, d_v, _strides3(k_strides), _strides3(v_strides),
                                       _stream(stream)), "moa_kv_append_strided")


def moa_decode_step_strided(q, K, V, k_new, v_new, out, lens, batch, h_q, h_kv, n_max, d_k, d_v, scale,
                            k_strides, v_strides, workspace, workspace_bytes, stream=None):
    _check(lib().moa_decode_step_strided(_ptr(q), _ptr(K), _ptr(V), _ptr(k_new), _ptr(v_new), _ptr(out),
                                         _ptr(lens), batch, h_q, h_kv, n_max, d_k, d_v, scale,
                                         _strides3(k_strides), _strides3(v_strides), _ptr(workspace),
                                         workspace_bytes, _stream(stream)), "moa_decode_step_strided")


def moa_decode_attn_host(q, K, V, out, batch, h_q, h_kv, n, d_k, d_v, scale):
    """q, K, V, out are HOST buffers (pinned tensors or numpy arrays)."""
    _check(lib().moa_decode_attn_host(_ptr(q), _ptr(K), _ptr(V), _ptr(out), batch, h_q, h_kv, n,
                                      d_k, d_v, scale), "moa_decode_attn_host")


def moa_device_status(stream=None) -> int:
    v = C.c_int(0)
    _check(lib().moa_device_status(_stream(stream), C.byref(v)), "moa_device_status")
    return v.value


def moa_min_bytes(batch, h_q, h_kv, n, d_k, d_v) -> int:
    return int(lib().moa_min_bytes(batch, h_q, h_kv, n, d_k, d_v))


def moa_release():
    _check(lib().moa_release(), "moa_release")


def moa_strerror(code: int) -> str:
    return strerror(code)


def moa_set_option(option: int, value: int):
    _check(lib().moa_set_option(option, value), "moa_set_option")


def moa_last_path() -> int:
    return int(lib().moa_last_path())


def moa_profile(enable: int):
    _check(lib().moa_profile(int(enable)), "moa_profile")


def moa_profile_read():
    """-> (decode_kernel_ms, decode_kernel_launches_timed, all_kernel_launches)."""
    ms, n, a = C.c_double(0), C.c_longlong(0), C.c_longlong(0)
    _check(lib().moa_profile_read(C.byref(ms), C.byref(n), C.byref(a)), "moa_profile_read")
    return ms.value, n.value, a.value


def moa_profile_launch_ms(index: int) -> float:
    """Event time of the index-th timed decode-kernel launch, in milliseconds."""
    ms = C.c_double(0)
    _check(lib().moa_profile_launch_ms(int(index), C.byref(ms)), "moa_profile_launch_ms")
    return ms.value

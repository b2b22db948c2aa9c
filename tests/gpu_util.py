"""Helpers for the GPU parity tests: device buffers with guard bands, calls through the
C ABI binding, comparison against the CPU oracle."""
import numpy as np
import torch

import paper_2607_19456_b200 as moa

TOL = 5e-6            # max abs error allowed for fp32 outputs against the fp64 oracle
GUARD = 64            # floats of guard band on each side (256 bytes keeps 16-byte alignment)
CANARY = 0x7FA5A5A5   # a NaN bit pattern: any use of it poisons the result


class Guarded:
    """A device tensor of `shape` (float32 or int32) surrounded by canary words.
    `misalign` shifts the payload by that many 4-byte words (to test unaligned pointers)."""

    def __init__(self, host=None, shape=None, dtype=np.float32, misalign=0, fill=None):
        if host is not None:
            host = np.ascontiguousarray(host)
            shape, dtype = host.shape, host.dtype
        self.shape, self.dtype = tuple(shape), np.dtype(dtype)
        self.n = int(np.prod(self.shape))
        self.off = GUARD + misalign
        total = self.n + 2 * GUARD + misalign
        raw = np.full(total, CANARY, np.uint32)
        if host is not None:
            raw[self.off:self.off + self.n] = host.reshape(-1).view(np.uint32)
        elif fill is not None:
            raw[self.off:self.off + self.n] = np.full(self.n, fill, self.dtype).view(np.uint32)
        self.raw = torch.from_numpy(raw.view(np.int32)).cuda()
        self.ptr = self.raw.data_ptr() + 4 * self.off

    def host(self):
        r = self.raw.cpu().numpy().view(np.uint32)
        return r[self.off:self.off + self.n].view(self.dtype).reshape(self.shape).copy()

    def guards_intact(self):
        r = self.raw.cpu().numpy().view(np.uint32)
        return bool(np.all(r[:self.off] == CANARY) and np.all(r[self.off + self.n:] == CANARY))


def workspace_for(B, hq, hkv, n_max, dk, dv):
    nbytes = moa.moa_workspace_bytes(B, hq, hkv, n_max, dk, dv)
    g = Guarded(shape=((nbytes + 3) // 4,), dtype=np.float32)
    assert g.ptr % 256 == 0
    return g, nbytes


def gpu_decode(q, K, V, scale, seq_lens=None, misalign=0, path=moa.PATH_AUTO, num_ctas=0,
               expect_path=None):
    """Run the library on host arrays; returns out [B,h_q,d_v] (numpy).  Checks guard bands
    of every buffer and that the device status word stays clear."""
    B, hq, dk = q.shape
    _, hkv, n, _ = K.shape
    dv = V.shape[3]
    gq, gK, gV = Guarded(q, misalign=misalign), Guarded(K, misalign=misalign), Guarded(V, misalign=misalign)
    gout = Guarded(shape=(B, hq, dv), misalign=misalign)
    moa.moa_set_option(moa.OPT_FORCE_PATH, path)
    moa.moa_set_option(moa.OPT_NUM_CTAS, num_ctas)
    try:
        if seq_lens is None:
            moa.moa_decode_attn(gq.ptr, gK.ptr, gV.ptr, gout.ptr, B, hq, hkv, n, dk, dv, scale)
            bufs = (gq, gK, gV, gout)
        else:
            glens = Guarded(np.asarray(seq_lens, np.int32))
            gws, nbytes = workspace_for(B, hq, hkv, n, dk, dv)
            moa.moa_decode_attn_varlen(gq.ptr, gK.ptr, gV.ptr, gout.ptr, B, hq, hkv, glens.ptr, n,
                                       dk, dv, scale, gws.ptr, nbytes)
            bufs = (gq, gK, gV, gout, glens, gws)
        torch.cuda.synchronize()
        used = moa.moa_last_path()
    finally:
        moa.moa_set_option(moa.OPT_FORCE_PATH, 0)
        moa.moa_set_option(moa.OPT_NUM_CTAS, 0)
    assert moa.moa_device_status() == 0
    for g in bufs:
        assert g.guards_intact(), "a kernel wrote outside its buffer"
    if expect_path is not None:
        assert used == expect_path, "kernel path %d ran, expected %d" % (used, expect_path)
    return gout.host()


def max_err(a, b):
    return float(np.max(np.abs(a.astype(np.float64) - b.astype(np.float64))))

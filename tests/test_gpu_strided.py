"""GPU parity for caches that are not densely packed: batch, head and row strides given in
elements (moa_decode_attn_strided, moa_kv_append_strided, moa_decode_step_strided).  The
oracle always sees the dense copy of the addressed rows; the bytes between the rows hold a NaN
pattern on the device, so a kernel that reads a wrong address poisons its result, and they
must come back unchanged."""
import numpy as np
import pytest

import moa_inputs as mi
import oracle
import paper_2607_19456_b200 as moa
from gpu_util import CANARY, TOL, Guarded, max_err, workspace_for

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def strides_for(kind, B, h, n, d):
    """(batch, head, row) element strides of a [B, h, n, d] cache in layout `kind`."""
    if kind == "dense":
        return (h * n * d, n * d, d)
    if kind == "gap":                       # rows contiguous, padding between heads and between items
        sh = n * d + 20
        return (h * sh + 8, sh, d)
    if kind == "nhd":                       # [B, n, h, d]: heads innermost
        return (n * h * d, d, h * d)
    if kind == "nhd_pad":                   # the same with padded rows
        sr = h * d + 12
        return (n * sr + 4, d, sr)
    if kind == "bcast":                     # every batch item reads the same rows
        return (0, n * d, d)
    if kind == "odd":                       # strides that are not multiples of 16 bytes
        sr = d + 1
        return (h * n * sr + 3, n * sr, sr)
    raise ValueError(kind)


def place(dense, strides):
    """Flat uint32 image of `dense` [B,h,n,d] laid out with `strides`; gaps hold the canary."""
    B, h, n, d = dense.shape
    sb, sh, sr = strides
    size = (B - 1) * sb + (h - 1) * sh + (n - 1) * sr + d
    flat = np.full(size, CANARY, np.uint32)
    src = dense.view(np.uint32)
    for b in range(B):
        for hh in range(h):
            base = b * sb + hh * sh
            idx = base + (np.arange(n)[:, None] * sr + np.arange(d)[None, :])
            flat[idx.reshape(-1)] = src[b, hh].reshape(-1)
    return flat.view(np.float32)


def run_strided(kind, seed, B, hq, hkv, n, dk, dv, lens=None, expect=None, path=moa.PATH_AUTO):
    w = mi.Workload("t", seed, B, hq, hkv, n, dk, dv)
    q, K, V, s = w.q(), w.K(), w.V(), w.scale
    if kind == "bcast":
        K = np.ascontiguousarray(np.broadcast_to(K[:1], K.shape))
        V = np.ascontiguousarray(np.broadcast_to(V[:1], V.shape))
    ks, vs = strides_for(kind, B, hkv, n, dk), strides_for(kind, B, hkv, n, dv)
    gq, gK, gV = Guarded(q), Guarded(place(K, ks)), Guarded(place(V, vs))
    gout = Guarded(shape=(B, hq, dv))
    gws, nbytes = workspace_for(B, hq, hkv, n, dk, dv)
    glens = Guarded(np.asarray(lens, np.int32)) if lens is not None else None
    moa.moa_set_option(moa.OPT_FORCE_PATH, path)
    try:
        moa.moa_decode_attn_strided(gq.ptr, gK.ptr, gV.ptr, gout.ptr, glens.ptr if glens else None, B, hq, hkv,
                                    n, dk, dv, s, ks, vs, gws.ptr, nbytes)
        torch.cuda.synchronize()
        used = moa.moa_last_path()
    finally:
        moa.moa_set_option(moa.OPT_FORCE_PATH, 0)
    assert moa.moa_device_status() == 0
    for g in (gq, gK, gV, gout, gws) + ((glens,) if glens else ()):
        assert g.guards_intact()
    if expect is not None:
        assert used in expect, "kernel path %d ran, expected one of %s" % (used, expect)
    ref = oracle.decode(q, K, V, s) if lens is None else oracle.decode_varlen(q, K, V, np.asarray(lens, np.int32), s)
    assert max_err(gout.host(), ref) <= TOL, (kind, B, hq, hkv, n, dk, dv)
    return used


@pytest.mark.parametrize("kind", ["dense", "gap", "bcast"])
@pytest.mark.parametrize("D,gs", [(128, 1), (128, 4), (64, 2), (32, 4), (32, 8)])
def test_contiguous_rows_small_groups_run_on_the_fma_kernel(kind, D, gs):
    for n in (5, 300, 1037):
        run_strided(kind, 31 * D + gs + n, 3, 2 * gs, 2, n, D, D, expect=(moa.PATH_STREAM,))


@pytest.mark.parametrize("kind", ["dense", "gap"])
@pytest.mark.parametrize("D,gs", [(128, 8), (64, 8), (128, 12), (128, 16), (128, 64), (64, 24)])
def test_contiguous_rows_large_groups_run_on_the_mma_kernel(kind, D, gs):
    for n in (9, 700):
        tensor_core = kind == "dense" and ((D == 128 and gs == 64) or
                                           (D == 64 and gs == 24 and n % 2 == 0))     # rows of 64 features go in pairs
        run_strided(kind, 17 * D + gs + n, 2, 2 * gs, 2, n, D, D,
                    expect=(moa.PATH_GROUPED,) if tensor_core else (moa.PATH_MMA,))


@pytest.mark.parametrize("kind", ["nhd", "nhd_pad"])
@pytest.mark.parametrize("dk,dv,gs", [(128, 128, 1), (128, 128, 4), (128, 128, 8), (64, 64, 2), (64, 64, 16),
                                      (128, 64, 4), (64, 128, 8), (128, 128, 12), (128, 128, 32), (128, 128, 21),
                                      (64, 128, 19)])
def test_heads_innermost_runs_on_the_mma_kernel(kind, dk, dv, gs):
    for n in (1, 16, 17, 333, 1500):
        run_strided(kind, dk + 3 * dv + gs + n, 2, 3 * gs, 3, n, dk, dv, expect=(moa.PATH_MMA,))


@pytest.mark.parametrize("kind", ["nhd", "odd"])
def test_layouts_without_a_fast_kernel_run_on_the_catch_all_kernel(kind):
    run_strided(kind, 5, 2, 4, 2, 77, 32, 32, expect=(moa.PATH_GENERIC,))          # d = 32 with a row stride
    run_strided(kind, 6, 2, 4, 2, 77, 24, 40, expect=(moa.PATH_GENERIC,))
    if kind == "odd":
        run_strided(kind, 7, 2, 8, 2, 130, 128, 128, expect=(moa.PATH_GENERIC,))
    # 20 heads per group: virtual heads of 8, 8 and 4 on the warp-MMA kernel where tiled copies are possible
    run_strided(kind, 8, 2, 40, 2, 50, 128, 128, expect=(moa.PATH_GENERIC if kind == "odd" else moa.PATH_MMA,))


def test_shared_rows_for_every_batch_item_on_large_groups():
    # a zero batch stride on the kernel that addresses through tensor maps: whichever kernel
    # the library settles on, the answer is the dense one
    for gs in (8, 16):
        run_strided("bcast", 40 + gs, 3, 2 * gs, 2, 500, 128, 128,
                    expect=(moa.PATH_MMA, moa.PATH_GENERIC))


@pytest.mark.parametrize("kind", ["gap", "nhd", "nhd_pad", "odd"])
def test_ragged_lengths_with_strides(kind):
    rng = np.random.default_rng(3)
    for (hq, hkv, D) in ((8, 2, 128), (16, 2, 64), (4, 4, 128)):
        B, n = 5, 900
        lens = rng.integers(1, n + 1, size=B)
        lens[0], lens[1] = 1, n
        run_strided(kind, 90 + hq + D, B, hq, hkv, n, D, D, lens=lens)


def test_forced_fma_kernel_refuses_a_row_stride():
    with pytest.raises(moa.MoaError) as e:
        run_strided("nhd", 1, 2, 8, 2, 100, 128, 128, path=moa.PATH_STREAM)
    assert e.value.code == moa.ERR_UNSUPPORTED


def test_stride_validation():
    w = mi.Workload("t", 1, 2, 4, 2, 64, 64, 64)
    gq, gK, gV = Guarded(w.q()), Guarded(w.K()), Guarded(w.V())
    gout = Guarded(shape=(2, 4, 64))
    dense = strides_for("dense", 2, 2, 64, 64)
    for bad in ((-1, 64 * 64, 64), (2 * 64 * 64, 64 * 64, 63), (1 << 41, 64 * 64, 64)):
        for args in ((bad, dense), (dense, bad)):
            with pytest.raises(moa.MoaError) as e:
                moa.moa_decode_attn_strided(gq.ptr, gK.ptr, gV.ptr, gout.ptr, None, 2, 4, 2, 64, 64, 64, 0.125,
                                            args[0], args[1])
            assert e.value.code == moa.ERR_INVALID
    # a cache that is written may not alias itself
    glens = Guarded(np.zeros(2, np.int32))
    gws, nbytes = workspace_for(2, 4, 2, 64, 64, 64)
    knew = Guarded(np.zeros((2, 2, 64), np.float32))
    with pytest.raises(moa.MoaError) as e:
        moa.moa_decode_step_strided(gq.ptr, gK.ptr, gV.ptr, knew.ptr, knew.ptr, gout.ptr, glens.ptr, 2, 4, 2, 64,
                                    64, 64, 0.125, (0, 64 * 64, 64), dense, gws.ptr, nbytes)
    assert e.value.code == moa.ERR_INVALID
    with pytest.raises(moa.MoaError) as e:
        moa.moa_kv_append_strided(gK.ptr, gV.ptr, knew.ptr, knew.ptr, glens.ptr, 2, 2, 64, 64, 64, dense,
                                  (2 * 64 * 64, 0, 64))
    assert e.value.code == moa.ERR_INVALID
    torch.cuda.synchronize()
    assert gK.guards_intact() and gV.guards_intact() and gout.guards_intact()


@pytest.mark.parametrize("kind,hq,hkv,dk,dv,expect", [
    ("gap", 8, 2, 128, 128, moa.PATH_STREAM),
    ("gap", 16, 2, 64, 64, moa.PATH_MMA),
    ("nhd", 8, 2, 128, 128, moa.PATH_MMA),
    ("nhd_pad", 8, 1, 64, 128, moa.PATH_MMA),
    ("nhd", 4, 2, 32, 32, moa.PATH_GENERIC),
    ("odd", 6, 2, 128, 128, moa.PATH_GENERIC),
])
def test_decode_steps_on_a_strided_cache(kind, hq, hkv, dk, dv, expect):
    """Four autoregressive steps: outputs against the oracle, the cache image bit for bit
    (appended rows in place, every byte between the rows untouched), lengths advanced."""
    B, n_max, steps = 3, 40, 4
    w = mi.Workload("t", 77 + hq + dk, B, hq, hkv, n_max, dk, dv)
    K, V, s = w.K().copy(), w.V().copy(), w.scale
    lens = np.array([0, 17, n_max - steps], np.int32)
    ks, vs = strides_for(kind, B, hkv, n_max, dk), strides_for(kind, B, hkv, n_max, dv)
    gK, gV = Guarded(place(K, ks)), Guarded(place(V, vs))
    glens = Guarded(lens)
    gws, nbytes = workspace_for(B, hq, hkv, n_max, dk, dv)
    rng = np.random.default_rng(11)
    for t in range(steps):
        q = rng.standard_normal((B, hq, dk)).astype(np.float32)
        k_new = rng.standard_normal((B, hkv, dk)).astype(np.float32)
        v_new = rng.standard_normal((B, hkv, dv)).astype(np.float32)
        gq, gk, gv = Guarded(q), Guarded(k_new), Guarded(v_new)
        gout = Guarded(shape=(B, hq, dv))
        moa.moa_decode_step_strided(gq.ptr, gK.ptr, gV.ptr, gk.ptr, gv.ptr, gout.ptr, glens.ptr, B, hq, hkv,
                                    n_max, dk, dv, s, ks, vs, gws.ptr, nbytes)
        torch.cuda.synchronize()
        assert moa.moa_last_path() == expect
        assert moa.moa_device_status() == 0
        oracle.kv_append(K, V, k_new, v_new, lens)
        lens = lens + 1
        assert max_err(gout.host(), oracle.decode_varlen(q, K, V, lens, s)) <= TOL, (kind, t)
        assert np.array_equal(glens.host(), lens)
        for g in (gq, gk, gv, gout, gK, gV, glens, gws):
            assert g.guards_intact()
    assert np.array_equal(gK.host().view(np.uint32), place(K, ks).view(np.uint32))
    assert np.array_equal(gV.host().view(np.uint32), place(V, vs).view(np.uint32))


def test_append_on_a_strided_cache_is_bit_exact():
    B, hkv, n_max, dk, dv = 3, 2, 20, 24, 40
    w = mi.Workload("t", 5, B, 2, hkv, n_max, dk, dv)
    K, V = w.K(), w.V()
    for kind in ("gap", "nhd", "nhd_pad", "odd"):
        ks, vs = strides_for(kind, B, hkv, n_max, dk), strides_for(kind, B, hkv, n_max, dv)
        gK, gV = Guarded(place(K, ks)), Guarded(place(V, vs))
        pos = np.array([0, 7, n_max - 1], np.int32)
        rng = np.random.default_rng(2)
        k_new = rng.standard_normal((B, hkv, dk)).astype(np.float32)
        v_new = rng.standard_normal((B, hkv, dv)).astype(np.float32)
        k_new.view(np.uint32)[0, 0, 0] = 0x7FC12345       # NaN payloads travel as raw bits
        gk, gv, gpos = Guarded(k_new), Guarded(v_new), Guarded(pos)
        moa.moa_kv_append_strided(gK.ptr, gV.ptr, gk.ptr, gv.ptr, gpos.ptr, B, hkv, n_max, dk, dv, ks, vs)
        torch.cuda.synchronize()
        assert moa.moa_device_status() == 0
        K2, V2 = K.copy(), V.copy()
        oracle.kv_append(K2, V2, k_new, v_new, pos)
        assert np.array_equal(gK.host().view(np.uint32), place(K2, ks).view(np.uint32))
        assert np.array_equal(gV.host().view(np.uint32), place(V2, vs).view(np.uint32))
        assert gK.guards_intact() and gV.guards_intact()


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("gs", [1, 2, 3, 4, 7])
def test_small_groups_padded_to_eight_heads_on_the_mma_kernel(D, gs):
    # the configuration a row stride selects, forced on a dense cache as well
    for n in (3, 250, 2100):
        run_strided("dense", 7 * D + gs + n, 2, 2 * gs, 2, n, D, D, path=moa.PATH_MMA, expect=(moa.PATH_MMA,))

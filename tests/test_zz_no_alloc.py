"""The allocation-free decode entry point, for callers that cannot call cudaMalloc (all
device memory already owned by a framework's pool, or a serving loop that must not take
the device-wide stall an allocation causes).  It must give what the ordinary entry point
gives, on consecutive calls that share the library's fixed scratch array.

This file sorts last on purpose: a run that stops at the first failure has then already
run every other test."""
import numpy as np
import pytest

import moa_inputs as mi
import paper_2607_19456_b200 as moa

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

TOL = 5e-6


def both_entry_points(w):
    q, K, V = (torch.from_numpy(x).cuda() for x in (w.q(), w.K(), w.V()))
    args = (w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale)
    ref = torch.full((w.batch, w.h_q, w.d_v), float("nan"), device="cuda")
    got = torch.full((w.batch, w.h_q, w.d_v), float("nan"), device="cuda")
    moa.moa_decode_attn(q, K, V, ref, *args)
    assert moa.moa_last_path() in (moa.PATH_STREAM, moa.PATH_MMA)    # the kernels that use scratch
    moa.moa_decode_attn_noalloc(q, K, V, got, *args)
    assert moa.moa_last_path() in (moa.PATH_STREAM, moa.PATH_MMA)
    torch.cuda.synchronize()
    assert moa.moa_device_status() == 0
    return ref.cpu().numpy(), got.cpu().numpy()


def test_noalloc_matches_the_allocating_entry_point_twice_in_a_row():
    # first a large problem that fills many scratch slots, then a smaller one of another
    # shape that finds the first call's leftovers in the array
    first = mi.Workload("na1", 4101, 3, 32, 8, 6000, 128, 128)
    second = mi.Workload("na2", 4102, 2, 16, 1, 1777, 64, 64)
    for w in (first, second):
        ref, got = both_entry_points(w)
        assert np.all(np.isfinite(got))
        assert float(np.max(np.abs(got.astype(np.float64) - ref.astype(np.float64)))) <= TOL


def test_noalloc_rejects_a_scratch_need_beyond_the_fixed_array():
    w = mi.Workload("na3", 4103, 1, 8, 1, 64, 128, 128)
    q, K, V = (torch.from_numpy(x).cuda() for x in (w.q(), w.K(), w.V()))
    out = torch.full((w.batch, w.h_q, w.d_v), -7.0, device="cuda")
    moa.moa_set_option(moa.OPT_NUM_CTAS, 4000)              # 4000 CTAs * 2 slots * 8 heads > 2 MiB
    try:
        with pytest.raises(moa.MoaError) as e:
            moa.moa_decode_attn_noalloc(q, K, V, out, w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale)
    finally:
        moa.moa_set_option(moa.OPT_NUM_CTAS, 0)
    assert e.value.code == moa.ERR_CAPACITY
    torch.cuda.synchronize()
    assert bool((out == -7.0).all())                        # nothing was launched

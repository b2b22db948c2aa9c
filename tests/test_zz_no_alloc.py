"""The allocation-free decode entry point, for callers that cannot call cudaMalloc (all
device memory already owned by a framework's pool, or a serving loop that must not take
the device-wide stall an allocation causes).  It must give what the ordinary entry point
gives, on consecutive calls that share the library's fixed scratch array.

This file sorts last on purpose: a run that stops at the first failure has then already
run every other test."""
import numpy as np
import pytest

import moa_inputs as mi
import oracle
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
    moa.moa_decode_attn_noalloc(q, K, V, got, *args)
    assert moa.moa_last_path() in (moa.PATH_STREAM, moa.PATH_MMA)    # the kernels that use scratch
    torch.cuda.synchronize()
    assert moa.moa_device_status() == 0
    return ref.cpu().numpy(), got.cpu().numpy(), oracle.decode(w.q(), w.K(), w.V(), w.scale)


def err(a, b):
    return float(np.max(np.abs(a.astype(np.float64) - b.astype(np.float64))))


def test_noalloc_matches_the_allocating_entry_point_twice_in_a_row():
    # first a large problem that fills many scratch slots, then a smaller one of another
    # shape that finds the first call's leftovers in the array
    first = mi.Workload("na1", 4101, 3, 32, 8, 6000, 128, 128)
    second = mi.Workload("na2", 4102, 2, 16, 1, 1777, 64, 64)
    for w in (first, second):
        ref, got, want = both_entry_points(w)
        assert np.all(np.isfinite(got))
        assert err(got, ref) <= TOL          # the two entry points agree ...
        assert err(got, want) <= TOL         # ... and both with the CPU oracle
        assert err(ref, want) <= TOL


@pytest.mark.parametrize("hq,hkv,d", [(64, 1, 128), (32, 2, 128), (12, 1, 128), (128, 2, 64)])
def test_noalloc_serves_the_largest_plans(hq, hkv, d):
    # tiles of 16 heads at d = 128 need the most scratch per CTA (2.5 MB on 148 SMs): MQA with
    # 64 heads, groups of 16 and of 9..15, and the same at d = 64; twice in a row each
    w = mi.Workload("na4", 4110 + hq + d, 2, hq, hkv, 3000, d, d)
    for _ in range(2):
        ref, got, want = both_entry_points(w)
        assert err(got, want) <= TOL and err(got, ref) <= TOL


def test_noalloc_rejects_a_scratch_need_beyond_the_fixed_array():
    w = mi.Workload("na3", 4103, 1, 8, 1, 64, 128, 128)
    q, K, V = (torch.from_numpy(x).cuda() for x in (w.q(), w.K(), w.V()))
    out = torch.full((w.batch, w.h_q, w.d_v), -7.0, device="cuda")
    moa.moa_set_option(moa.OPT_NUM_CTAS, 4000)              # 4000 CTAs * 2 slots * 8 heads * 132 floats > 4 MiB
    try:
        with pytest.raises(moa.MoaError) as e:
            moa.moa_decode_attn_noalloc(q, K, V, out, w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale)
    finally:
        moa.moa_set_option(moa.OPT_NUM_CTAS, 0)
    assert e.value.code == moa.ERR_CAPACITY
    torch.cuda.synchronize()
    assert bool((out == -7.0).all())                        # nothing was launched

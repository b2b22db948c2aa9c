"""The five benchmark workloads at full size, in the launch configuration bench.py times
(default CTA count, library workspace), against the CPU oracle.  Where the oracle cannot
afford the whole tensor it recomputes sampled (batch, kv-head) groups one by one from
independently regenerated K/V slabs."""
import numpy as np
import pytest

import moa_inputs as mi
import oracle
import paper_2607_19456_b200 as moa
from gpu_util import TOL, max_err

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def run_dense_on_gpu(w):
    q, K, V = w.q(), w.K(), w.V()
    dq, dK, dV = torch.from_numpy(q).cuda(), torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda()
    del K, V
    out = torch.full((w.batch, w.h_q, w.d_v), float("nan"), device="cuda")
    moa.moa_decode_attn(dq, dK, dV, out, w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale)
    torch.cuda.synchronize()
    want = moa.PATH_STREAM
    if 17 <= w.group <= 64 and w.d_k == 128:
        want = moa.PATH_GROUPED
    elif 17 <= w.group <= 64 and w.d_k == 64 and w.n % 2 == 0:
        want = moa.PATH_GROUPED              # rows of 64 features, taken in pairs
    elif w.group % 8 == 0 and w.d_k >= 64:
        want = moa.PATH_MMA
    assert moa.moa_last_path() == want
    assert moa.moa_device_status() == 0
    res = out.cpu().numpy()
    del dq, dK, dV, out
    torch.cuda.empty_cache()
    return q, res


def check_units(w, q, res, units):
    g = w.group
    worst = 0.0
    for b, h in units:
        Ks, Vs = w.K_slab(b, h)[None, None], w.V_slab(b, h)[None, None]
        ref = oracle.decode(q[b:b + 1, h * g:(h + 1) * g], Ks, Vs, w.scale)
        worst = max(worst, max_err(res[b:b + 1, h * g:(h + 1) * g], ref))
    return worst


def sample_units(w, count, seed):
    r = np.random.default_rng(seed)
    units = {(0, 0), (w.batch - 1, w.h_kv - 1)}
    while len(units) < min(count, w.batch * w.h_kv):
        units.add((int(r.integers(w.batch)), int(r.integers(w.h_kv))))
    return sorted(units)


def test_config1_single_head_full():
    w = mi.WORKLOADS["single_head"]
    q, res = run_dense_on_gpu(w)
    assert max_err(res, oracle.decode(q, w.K(), w.V(), w.scale)) <= TOL


@pytest.mark.parametrize("name,count", [("mha", 16), ("gqa", 8), ("mqa_long", 2)])
def test_dense_configs_full_size_sampled(name, count):
    w = mi.WORKLOADS[name]
    q, res = run_dense_on_gpu(w)
    assert np.all(np.isfinite(res))
    assert check_units(w, q, res, sample_units(w, count, 5)) <= TOL


@pytest.mark.parametrize("name,count", [("extra_group8_d128", 6), ("extra_group8_d64", 6), ("extra_group16_d128", 6),
                                        ("extra_mha_d32", 12), ("extra_mqa_d64", 2)])
def test_extra_bench_shapes_full_size_sampled(name, count):
    # the timing-only shapes of bench.py (warp-MMA kernel at 8 and 16 heads per row, d = 32)
    import bench
    w = bench.EXTRA_WORKLOADS[name]
    q, res = run_dense_on_gpu(w)
    assert np.all(np.isfinite(res))
    assert check_units(w, q, res, sample_units(w, count, 6)) <= TOL


def test_config5_multi_step_full():
    w = mi.WORKLOADS["multi_step"]
    B, hq, hkv, n_max, d, T = w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.steps
    lens = w.start_lens()
    K, V = w.K(), w.V()
    for b in range(B):
        K[b, :, lens[b]:] = 0
        V[b, :, lens[b]:] = 0
    dK, dV = torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda()
    k_all = mi.normal(w.seed, mi.TID_KNEW, (T, B, hkv, d))
    v_all = mi.normal(w.seed, mi.TID_VNEW, (T, B, hkv, d))
    q_all = mi.normal(w.seed, mi.TID_QSTEP, (T, B, hq, d))
    assert np.array_equal(k_all[3], w.k_new(3)) and np.array_equal(q_all[7], w.q_step(7))
    dk, dv, dq = torch.from_numpy(k_all).cuda(), torch.from_numpy(v_all).cuda(), torch.from_numpy(q_all).cuda()
    dlens = torch.from_numpy(lens).cuda()
    nbytes = moa.moa_workspace_bytes(B, hq, hkv, n_max, d, d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    out = torch.empty((B, hq, d), device="cuda")
    checked = {0, 1, 2, 100, 255, 510, 511}
    worst = 0.0
    for t in range(T):
        moa.moa_decode_step(dq[t], dK, dV, dk[t], dv[t], out, dlens, B, hq, hkv, n_max, d, d, w.scale,
                            ws, nbytes)
        oracle.kv_append(K, V, k_all[t], v_all[t], lens)
        lens = lens + 1
        if t in checked:
            ref = oracle.decode_varlen(q_all[t], K, V, lens, w.scale)
            worst = max(worst, max_err(out.cpu().numpy(), ref))
    torch.cuda.synchronize()
    assert moa.moa_device_status() == 0
    assert worst <= TOL
    assert np.array_equal(dlens.cpu().numpy(), lens)
    assert np.array_equal(dK.cpu().numpy().view(np.uint32), K.view(np.uint32))
    assert np.array_equal(dV.cpu().numpy().view(np.uint32), V.view(np.uint32))

"""Seeded random shapes through every entry point of the decode path, against the oracle:
dense and ragged caches, plain decode and the fused append+decode step, every group size
from 1 to 64 and d in {32, 64, 128} (so every kernel family and every compiled
configuration is reached by several cases), odd batch and head counts, short and long rows."""
import numpy as np
import pytest

import moa_inputs as mi
import oracle
import paper_2607_19456_b200 as moa
from gpu_util import TOL, Guarded, gpu_decode, max_err, workspace_for

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

GROUPS = [1, 2, 3, 4, 5, 6, 7, 8, 8, 9, 12, 16, 16, 19, 20, 24, 27, 32, 43, 48, 63, 64]


def draw(case):
    r = np.random.default_rng(9000 + case)
    d = int(r.choice([32, 64, 128]))
    gs = int(r.choice(GROUPS))
    hkv = int(r.integers(1, 4))
    B = int(r.integers(1, 5))
    n = int(r.choice([1, 2, 15, 16, 17, 31, 33, 100, 257, 1000, 2049, int(r.integers(1, 3000))]))
    return r, B, gs * hkv, hkv, n, d


@pytest.mark.parametrize("case", range(48))
def test_random_dense_and_ragged(case):
    r, B, hq, hkv, n, d = draw(case)
    q = mi.normal(9000 + case, 1, (B, hq, d))
    K = mi.normal(9000 + case, 2, (B, hkv, n, d))
    V = mi.normal(9000 + case, 3, (B, hkv, n, d))
    s = 1.0 / np.sqrt(d)
    assert max_err(gpu_decode(q, K, V, s), oracle.decode(q, K, V, s)) <= TOL, (B, hq, hkv, n, d)
    lens = r.integers(1, n + 1, size=B).astype(np.int32)
    assert max_err(gpu_decode(q, K, V, s, seq_lens=lens), oracle.decode_varlen(q, K, V, lens, s)) <= TOL


@pytest.mark.parametrize("case", range(48, 80))
def test_random_fused_steps(case):
    r, B, hq, hkv, n_max, d = draw(case)
    n_max += 3
    w = mi.Workload("fz", 9000 + case, B, hq, hkv, n_max, d, d)
    K, V = w.K(), w.V()
    lens = r.integers(0, n_max - 2, size=B).astype(np.int32)
    gK, gV, glens = Guarded(K), Guarded(V), Guarded(lens)
    gws, nbytes = workspace_for(B, hq, hkv, n_max, d, d)
    gout = Guarded(shape=(B, hq, d))
    for t in range(3):
        kn, vn, qt = w.k_new(t), w.v_new(t), w.q_step(t)
        gk, gv, gq = Guarded(kn), Guarded(vn), Guarded(qt)
        moa.moa_decode_step(gq.ptr, gK.ptr, gV.ptr, gk.ptr, gv.ptr, gout.ptr, glens.ptr, B, hq, hkv, n_max, d, d,
                            w.scale, gws.ptr, nbytes)
        oracle.kv_append(K, V, kn, vn, lens)
        lens = lens + 1
        assert max_err(gout.host(), oracle.decode_varlen(qt, K, V, lens, w.scale)) <= TOL, (B, hq, hkv, n_max, d, t)
    assert moa.moa_device_status() == 0
    assert np.array_equal(glens.host(), lens)
    assert np.array_equal(gK.host().view(np.uint32), K.view(np.uint32))
    assert np.array_equal(gV.host().view(np.uint32), V.view(np.uint32))
    for g in (gK, gV, glens, gws, gout):
        assert g.guards_intact()


@pytest.mark.parametrize("case", range(24))
def test_random_large_groups_at_d64(case):
    """17..64 heads per K/V head on rows of 64 features: even capacities take the 64-lane
    tensor-core kernel two rows at a time (dense, ragged and fused step), odd ones the streaming
    kernels; both against the oracle."""
    r = np.random.default_rng(77000 + case)
    gs = int(r.choice([17, 18, 23, 24, 31, 32, 33, 41, 48, 63, 64])); hkv = int(r.integers(1, 4)); B = int(r.integers(1, 6))
    n = int(r.choice([2, 4, 16, 30, 128, 130, 254, 256, 258, 1000, 2050, 2 * int(r.integers(1, 2500)), int(r.integers(1, 3000))]))
    hq = gs * hkv
    q = mi.normal(77000 + case, 1, (B, hq, 64))
    K = mi.normal(77000 + case, 2, (B, hkv, n, 64))
    V = mi.normal(77000 + case, 3, (B, hkv, n, 64))
    assert max_err(gpu_decode(q, K, V, 0.125), oracle.decode(q, K, V, 0.125)) <= TOL, (B, hq, hkv, n)
    lens = r.integers(1, n + 1, size=B).astype(np.int32)
    assert max_err(gpu_decode(q, K, V, 0.125, seq_lens=lens), oracle.decode_varlen(q, K, V, lens, 0.125)) <= TOL
    n_max = n + 4
    w = mi.Workload("fzp", 77000 + case, B, hq, hkv, n_max, 64, 64)
    K, V = w.K(), w.V()
    lens = r.integers(0, n_max - 3, size=B).astype(np.int32)
    gK, gV, glens = Guarded(K), Guarded(V), Guarded(lens)
    gws, nbytes = workspace_for(B, hq, hkv, n_max, 64, 64)
    gout = Guarded(shape=(B, hq, 64))
    for t in range(3):
        kn, vn, qt = w.k_new(t), w.v_new(t), w.q_step(t)
        gk, gv, gq = Guarded(kn), Guarded(vn), Guarded(qt)
        moa.moa_decode_step(gq.ptr, gK.ptr, gV.ptr, gk.ptr, gv.ptr, gout.ptr, glens.ptr, B, hq, hkv, n_max, 64, 64,
                            w.scale, gws.ptr, nbytes)
        oracle.kv_append(K, V, kn, vn, lens)
        lens = lens + 1
        assert max_err(gout.host(), oracle.decode_varlen(qt, K, V, lens, w.scale)) <= TOL, (B, hq, hkv, n_max, t)
    assert moa.moa_device_status() == 0
    assert np.array_equal(gK.host().view(np.uint32), K.view(np.uint32))
    assert np.array_equal(gV.host().view(np.uint32), V.view(np.uint32))
    for g in (gK, gV, glens, gws, gout):
        assert g.guards_intact()

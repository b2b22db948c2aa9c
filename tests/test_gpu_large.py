"""Caches of more than 2^32 elements each (18 GB of K and 18 GB of V): every kernel family's
address arithmetic beyond 32 bits.  The caches are filled on the device by a seeded
generator; the oracle recomputes sampled (batch, kv-head) groups from slabs copied back:
the first and last group and the groups on either side of element 2^31 and of element 2^32."""
import numpy as np
import pytest

import oracle
import paper_2607_19456_b200 as moa
from gpu_util import TOL, max_err

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

B, H_KV, N, D = 136, 8, 32768, 128            # 136*8*32768*128 = 4.56e9 elements per cache
UNIT = N * D                                  # elements per (batch, kv head)
SCALE = 1.0 / np.sqrt(D)
EDGES = [0, (1 << 31) // UNIT - 1, (1 << 31) // UNIT, (1 << 32) // UNIT - 1, (1 << 32) // UNIT, B * H_KV - 1]


@pytest.fixture(scope="module")
def caches():
    free, _ = torch.cuda.mem_get_info()
    need = 2 * B * H_KV * UNIT * 4
    if free < need + (4 << 30):
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    assert B * H_KV * UNIT > (1 << 32)
    g = torch.Generator(device="cuda").manual_seed(20260719)
    K = torch.empty((B, H_KV, N, D), device="cuda")
    V = torch.empty((B, H_KV, N, D), device="cuda")
    for t in (K, V):
        for b in range(0, B, 8):              # the generator's temporaries stay small
            t[b:b + 8].normal_(generator=g)
    yield K, V
    del K, V
    torch.cuda.empty_cache()


def units_to_check(extra_seed):
    r = np.random.default_rng(extra_seed)
    return sorted(set(EDGES) | {int(r.integers(B * H_KV)) for _ in range(2)})


def queries(h_q, seed):
    return np.random.default_rng(seed).standard_normal((B, h_q, D)).astype(np.float32)


def check_decode(K, V, q, res, g_s, lens=None, units=None):
    worst = 0.0
    for u in units:
        b, h = divmod(u, H_KV)
        n = N if lens is None else int(lens[b])
        Ks = K[b, h, :n].cpu().numpy()[None, None]
        Vs = V[b, h, :n].cpu().numpy()[None, None]
        ref = oracle.decode(q[b:b + 1, h * g_s:(h + 1) * g_s], Ks, Vs, SCALE)
        worst = max(worst, max_err(res[b:b + 1, h * g_s:(h + 1) * g_s], ref))
    return worst


@pytest.mark.parametrize("g_s,path", [(1, "PATH_STREAM"), (8, "PATH_MMA"), (64, "PATH_GROUPED")])
def test_dense_decode_over_caches_beyond_32_bit_offsets(caches, g_s, path):
    K, V = caches
    h_q = H_KV * g_s
    q = queries(h_q, 7 + g_s)
    dq = torch.from_numpy(q).cuda()
    out = torch.full((B, h_q, D), float("nan"), device="cuda")
    moa.moa_decode_attn(dq, K, V, out, B, h_q, H_KV, N, D, D, SCALE)
    torch.cuda.synchronize()
    assert moa.moa_last_path() == getattr(moa, path)
    assert moa.moa_device_status() == 0
    res = out.cpu().numpy()
    assert np.all(np.isfinite(res))
    assert check_decode(K, V, q, res, g_s, units=units_to_check(g_s)) <= TOL


@pytest.mark.parametrize("g_s", [1, 8, 64])
def test_fused_step_appends_and_attends_beyond_32_bit_offsets(caches, g_s):
    K, V = caches
    h_q = H_KV * g_s
    r = np.random.default_rng(100 + g_s)
    lens0 = r.integers(N // 2, N - 1, size=B).astype(np.int32)
    lens0[-1] = N - 1                          # the very last row of the cache gets written
    q = queries(h_q, 17 + g_s)
    k_new = r.standard_normal((B, H_KV, D)).astype(np.float32)
    v_new = r.standard_normal((B, H_KV, D)).astype(np.float32)
    units = units_to_check(50 + g_s)
    # what must not change: the row before and the row after the appended one
    before = {u: (K[u // H_KV, u % H_KV, lens0[u // H_KV] - 1].clone(), V[u // H_KV, u % H_KV, lens0[u // H_KV] - 1].clone())
              for u in units}
    after = {u: K[u // H_KV, u % H_KV, lens0[u // H_KV] + 1].clone() for u in units if lens0[u // H_KV] + 1 < N}
    dq, dk, dv = torch.from_numpy(q).cuda(), torch.from_numpy(k_new).cuda(), torch.from_numpy(v_new).cuda()
    dlens = torch.from_numpy(lens0.copy()).cuda()
    out = torch.full((B, h_q, D), float("nan"), device="cuda")
    nbytes = moa.moa_workspace_bytes(B, h_q, H_KV, N, D, D)
    ws = torch.empty((nbytes + 3) // 4, dtype=torch.float32, device="cuda")
    moa.moa_decode_step(dq, K, V, dk, dv, out, dlens, B, h_q, H_KV, N, D, D, SCALE, ws, nbytes)
    torch.cuda.synchronize()
    assert moa.moa_device_status() == 0
    assert np.array_equal(dlens.cpu().numpy(), lens0 + 1)
    for u in units:
        b, h = divmod(u, H_KV)
        p = int(lens0[b])
        assert np.array_equal(K[b, h, p].cpu().numpy().view(np.uint32), k_new[b, h].view(np.uint32))
        assert np.array_equal(V[b, h, p].cpu().numpy().view(np.uint32), v_new[b, h].view(np.uint32))
        assert torch.equal(K[b, h, p - 1], before[u][0]) and torch.equal(V[b, h, p - 1], before[u][1])
        if u in after:
            assert torch.equal(K[b, h, p + 1], after[u])
    res = out.cpu().numpy()
    assert np.all(np.isfinite(res))
    assert check_decode(K, V, q, res, g_s, lens=lens0 + 1, units=units) <= TOL


def test_strided_view_of_a_cache_beyond_32_bit_offsets(caches):
    # the same memory read as [B, N, H_KV, D] (heads innermost): element strides beyond 2^31
    K, V = caches
    g_s, h_q = 8, H_KV * 8
    q = queries(h_q, 31)
    dq = torch.from_numpy(q).cuda()
    out = torch.full((B, h_q, D), float("nan"), device="cuda")
    st = (H_KV * UNIT, D, H_KV * D)            # (batch, head, row) strides of the heads-innermost view
    n_view = N                                 # rows of that view per (batch, head)
    moa.moa_decode_attn_strided(dq, K, V, out, None, B, h_q, H_KV, n_view, D, D, SCALE, st, st)
    torch.cuda.synchronize()
    assert moa.moa_device_status() == 0
    res = out.cpu().numpy()
    Kv, Vv = K.view(B, N, H_KV, D), V.view(B, N, H_KV, D)
    worst = 0.0
    for u in units_to_check(77):
        b, h = divmod(u, H_KV)
        Ks = Kv[b, :, h].contiguous().cpu().numpy()[None, None]
        Vs = Vv[b, :, h].contiguous().cpu().numpy()[None, None]
        ref = oracle.decode(q[b:b + 1, h * g_s:(h + 1) * g_s], Ks, Vs, SCALE)
        worst = max(worst, max_err(res[b:b + 1, h * g_s:(h + 1) * g_s], ref))
    assert worst <= TOL

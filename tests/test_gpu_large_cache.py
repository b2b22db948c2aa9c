"""Caches whose tensors exceed 2^32 elements (and 2^32 bytes, several times over): the index
arithmetic of every kernel family, checked against the oracle on (batch, kv-head) units on
both sides of the 32-bit boundaries.  The cache is drawn on the device (seeded); the oracle
gets the sampled units' slabs copied back."""
import numpy as np
import pytest

import oracle
import paper_2607_19456_b200 as moa
from gpu_util import TOL, max_err

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

B, HKV, N, D = 136, 8, 32768, 128              # 4.56e9 floats = 18.3 GB per tensor; a slab is 16 MiB
# unit 255 ends at byte 2^32, unit 511 at element 2^31, unit 1023 at element 2^32
UNITS = [(0, 0), (31, 7), (32, 0), (63, 7), (64, 0), (127, 7), (128, 0), (135, 7)]


@pytest.fixture(scope="module")
def cache():
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2**30:
        pytest.skip("needs 60 GB of free device memory")
    g = torch.Generator(device="cuda").manual_seed(20260719)
    K = torch.randn((B, HKV, N, D), device="cuda", generator=g)
    V = torch.rand((B, HKV, N, D), device="cuda", generator=g)
    V.mul_(2.0).sub_(1.0)
    yield K, V, g
    del K, V
    torch.cuda.empty_cache()


def check(q, K, V, out, h_q, n, d, scale, lens=None):
    """Sampled units of `out` against the oracle; K, V viewed as [B, HKV, n, d]."""
    gs = h_q // HKV
    Kv, Vv = K.view(B, HKV, n, d), V.view(B, HKV, n, d)
    qh, oh = q.cpu().numpy(), out.cpu().numpy()
    assert np.all(np.isfinite(oh))
    worst = 0.0
    for b, h in UNITS:
        Ks, Vs = Kv[b, h].cpu().numpy()[None, None], Vv[b, h].cpu().numpy()[None, None]
        qs = qh[b:b + 1, h * gs:(h + 1) * gs]
        if lens is None:
            ref = oracle.decode(qs, Ks, Vs, scale)
        else:
            ref = oracle.decode_varlen(qs, Ks, Vs, np.asarray(lens[b:b + 1], np.int32), scale)
        worst = max(worst, max_err(oh[b:b + 1, h * gs:(h + 1) * gs], ref))
    return worst


@pytest.mark.parametrize("name,h_q,d,path", [
    ("fma_d128", 32, 128, moa.PATH_STREAM), ("mma_d128", 64, 128, moa.PATH_MMA),
    ("mma16_d128", 128, 128, moa.PATH_MMA), ("tcgen05_d128", 256, 128, moa.PATH_GROUPED),
    ("tcgen05_64heads_d128", 512, 128, moa.PATH_GROUPED),
    ("fma_d64", 16, 64, moa.PATH_STREAM), ("mma_d64", 64, 64, moa.PATH_MMA),
    ("tcgen05_pair_d64", 256, 64, moa.PATH_GROUPED), ("fma_d32", 8, 32, moa.PATH_STREAM)])
def test_dense_decode_on_a_cache_beyond_32_bit_offsets(cache, name, h_q, d, path):
    K, V, g = cache
    n = N * D // d                               # the same memory, rows of d features
    q = torch.randn((B, h_q, d), device="cuda", generator=g)
    out = torch.full((B, h_q, d), float("nan"), device="cuda")
    scale = 1.0 / np.sqrt(d)
    moa.moa_decode_attn(q, K, V, out, B, h_q, HKV, n, d, d, scale)
    torch.cuda.synchronize()
    assert moa.moa_last_path() == path and moa.moa_device_status() == 0
    assert check(q, K, V, out, h_q, n, d, scale) <= TOL


def test_generic_kernel_on_a_cache_beyond_32_bit_offsets(cache):
    K, V, g = cache
    q = torch.randn((B, HKV, D), device="cuda", generator=g)
    out = torch.full((B, HKV, D), float("nan"), device="cuda")
    moa.moa_set_option(moa.OPT_FORCE_PATH, moa.PATH_GENERIC)
    try:
        moa.moa_decode_attn(q, K, V, out, B, HKV, HKV, N, D, D, 0.09)
    finally:
        moa.moa_set_option(moa.OPT_FORCE_PATH, 0)
    torch.cuda.synchronize()
    assert moa.moa_last_path() == moa.PATH_GENERIC and moa.moa_device_status() == 0
    assert check(q, K, V, out, HKV, N, D, 0.09) <= TOL


@pytest.mark.parametrize("h_q", [32, 64, 256])
def test_ragged_lengths_on_a_cache_beyond_32_bit_offsets(cache, h_q):
    K, V, g = cache
    r = np.random.default_rng(11)
    lens = r.integers(1, N + 1, size=B).astype(np.int32)
    lens[[0, 31, 32, 63, 64, 127, 128, 135]] = [N, 1, N - 1, 4097, 129, N, 77, N]
    dl = torch.from_numpy(lens).cuda()
    q = torch.randn((B, h_q, D), device="cuda", generator=g)
    out = torch.full((B, h_q, D), float("nan"), device="cuda")
    nbytes = moa.moa_workspace_bytes(B, h_q, HKV, N, D, D)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    moa.moa_decode_attn_varlen(q, K, V, out, B, h_q, HKV, dl, N, D, D, 0.09, ws, nbytes)
    torch.cuda.synchronize()
    assert moa.moa_device_status() == 0
    assert check(q, K, V, out, h_q, N, D, 0.09, lens=lens) <= TOL


@pytest.mark.parametrize("h_q", [32, 64, 256])
def test_append_and_fused_step_on_a_cache_beyond_32_bit_offsets(cache, h_q):
    """The appended rows land where they belong (bit for bit, neighbours untouched) in units on
    both sides of the boundaries, and the step attends over them."""
    K, V, g = cache
    r = np.random.default_rng(12)
    lens = r.integers(1, N, size=B).astype(np.int32)
    lens[[0, 31, 32, 63, 64, 127, 128, 135]] = [N - 1, 1, N - 2, 4096, 128, N - 1, 77, N - 1]
    dl = torch.from_numpy(lens).cuda()
    k_new = torch.randn((B, HKV, D), device="cuda", generator=g)
    v_new = torch.randn((B, HKV, D), device="cuda", generator=g) + 3.0      # visible in the outputs, yet O(1): the bar is absolute
    q = torch.randn((B, h_q, D), device="cuda", generator=g)
    out = torch.full((B, h_q, D), float("nan"), device="cuda")
    before = {(b, h): (K[b, h, lens[b] - 1:lens[b] + 2].clone(), V[b, h, lens[b] - 1:lens[b] + 2].clone()) for b, h in UNITS}
    nbytes = moa.moa_workspace_bytes(B, h_q, HKV, N, D, D)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    moa.moa_decode_step(q, K, V, k_new, v_new, out, dl, B, h_q, HKV, N, D, D, 0.09, ws, nbytes)
    torch.cuda.synchronize()
    assert moa.moa_device_status() == 0
    assert np.array_equal(dl.cpu().numpy(), lens + 1)
    for (b, h), (kb, vb) in before.items():
        ka, va = K[b, h, lens[b] - 1:lens[b] + 2], V[b, h, lens[b] - 1:lens[b] + 2]
        assert torch.equal(ka[1].view(torch.int32), k_new[b, h].view(torch.int32))
        assert torch.equal(va[1].view(torch.int32), v_new[b, h].view(torch.int32))
        for i in (0, 2):
            if i < ka.shape[0]:
                assert torch.equal(ka[i].view(torch.int32), kb[i].view(torch.int32))
                assert torch.equal(va[i].view(torch.int32), vb[i].view(torch.int32))
    assert check(q, K, V, out, h_q, N, D, 0.09, lens=lens + 1) <= TOL

"""Pins for the CPU oracle: values the paper prints, closed forms, invariants, library
routines and an independent brute force.  No GPU.  Each check is chosen so that a
plausible slip in the oracle (dropped scale, wrong sign in the exponent, transposed
operand, wrong head mapping, off-by-one in the append offset) fails at least one."""
import math
from decimal import Decimal, getcontext

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import moa_inputs as mi
import oracle

getcontext().prec = 60


# --------------------------------------------------------------------------------------
# independent brute force: the *conventional* formulation (materialised transpose,
# softmax without max-subtraction) in 60-digit decimal arithmetic, pure Python.
# --------------------------------------------------------------------------------------
def brute_one_head(q, K, V, scale):
    n, d_k, d_v = len(K), len(q), len(V[0])
    qd = [Decimal(float(x)) for x in q]
    KT = [[Decimal(float(K[l][j])) for l in range(n)] for j in range(d_k)]   # K^T, d_k x n
    sc = Decimal(float(scale))
    scores = [sc * sum(qd[j] * KT[j][l] for j in range(d_k)) for l in range(n)]
    w = [s.exp() for s in scores]
    tot = sum(w)
    w = [x / tot for x in w]
    return [float(sum(w[l] * Decimal(float(V[l][d])) for l in range(n))) for d in range(d_v)]


def brute(q, K, V, scale):
    """q [B,hq,dk], K [B,hkv,n,dk], V [B,hkv,n,dv]; GQA by physically replicating K/V."""
    B, hq, _ = q.shape
    g = hq // K.shape[1]
    Kx, Vx = np.repeat(K, g, axis=1), np.repeat(V, g, axis=1)
    return np.array([[brute_one_head(q[b, h], Kx[b, h], Vx[b, h], scale)
                      for h in range(hq)] for b in range(B)])


def rnd(shape, seed, dist="normal"):
    r = np.random.default_rng(seed)
    x = r.standard_normal(shape) if dist == "normal" else r.uniform(-1, 1, shape)
    return x.astype(np.float32)


# --------------------------------------------------------------------------------------
# the paper's worked example
# --------------------------------------------------------------------------------------
def test_worked_example_printed_values(golden):
    g = golden("decode_example.txt")
    q = np.array(g["q"], np.float32).reshape(1, 1, 2)
    K = np.array(g["K"], np.float32).reshape(1, 1, 2, 2)
    V = np.array(g["V"], np.float32).reshape(1, 1, 2, 2)
    scale = 1.0 / math.sqrt(float(g["scale_is_inverse_sqrt_of"][0][0]))
    out = oracle.decode(q, K, V, scale)[0, 0]
    want = np.array(g["out"][0], float)
    # the paper prints two decimals and forms them from three-decimal weights
    assert np.all(np.abs(out - want) < 6e-3)
    # tighter: rebuild `out` from the paper's printed weights; must agree to their precision
    a = np.array(g["a"][0], float)
    assert np.all(np.abs(out - a @ V[0, 0].astype(float)) < 2e-3 * 8)
    # intermediate values printed by the paper, recovered from the oracle's output:
    # out = a0*V0 + (1-a0)*V1  =>  a0 = (V1 - out)/(V1 - V0)
    a0 = (6.0 - out[0]) / (6.0 - 2.0)
    assert abs(a0 - a[0]) < 5e-4 and abs((1 - a0) - a[1]) < 5e-4
    e1 = (1 - a0) / a0                       # e[1]/e[0] with e[0] = 1
    assert abs(e1 - float(g["e"][0][1])) < 5e-4
    assert abs((1 + e1) - float(g["Z"][0][0])) < 5e-4
    assert abs(-math.log(e1) - float(g["s"][0][0])) < 1e-6    # s[0]-s[1] = 1/sqrt 2


# --------------------------------------------------------------------------------------
# closed forms and invariants
# --------------------------------------------------------------------------------------
def test_n_equals_one_returns_v0_exactly():
    q, K, V = rnd((2, 4, 5), 1), rnd((2, 2, 1, 5), 2), rnd((2, 2, 1, 3), 3)
    out = oracle.decode(q, K, V, 0.37)
    want = np.repeat(V[:, :, 0, :], 2, axis=1)
    assert np.array_equal(out, want)


@pytest.mark.parametrize("case", ["identical_keys", "zero_query", "zero_scale"])
def test_uniform_weights_give_mean_of_V(case):
    n, dk, dv = 37, 6, 5
    q, K, V = rnd((1, 2, dk), 4), rnd((1, 1, n, dk), 5), rnd((1, 1, n, dv), 6)
    scale = 0.8
    if case == "identical_keys":
        K[:] = K[:, :, :1, :]
    elif case == "zero_query":
        q[:] = 0
    else:
        scale = 0.0
    out = oracle.decode(q, K, V, scale)
    mean = V[0, 0].astype(np.float64).mean(axis=0)
    assert np.allclose(out[0, 0], mean, rtol=0, atol=1e-7)
    assert np.allclose(out[0, 1], mean, rtol=0, atol=1e-7)


def test_shift_of_all_keys_leaves_output_unchanged():
    n, dk, dv = 50, 8, 7
    q, K, V = (rnd((1, 1, dk), 7).astype(np.float64), rnd((1, 1, n, dk), 8).astype(np.float64),
               rnd((1, 1, n, dv), 9).astype(np.float64))
    u = np.random.default_rng(10).standard_normal(dk)
    a = oracle.decode_f64(q, K, V, 0.5)
    b = oracle.decode_f64(q, K + u, V, 0.5)
    assert np.allclose(a, b, rtol=0, atol=1e-12)


def test_joint_row_permutation_leaves_output_unchanged():
    n, dk, dv = 64, 8, 9
    q, K, V = (rnd((1, 1, dk), 11).astype(np.float64), rnd((1, 1, n, dk), 12).astype(np.float64),
               rnd((1, 1, n, dv), 13).astype(np.float64))
    p = np.random.default_rng(14).permutation(n)
    a = oracle.decode_f64(q, K, V, 0.4)
    b = oracle.decode_f64(q, K[:, :, p], V[:, :, p], 0.4)
    assert np.allclose(a, b, rtol=0, atol=1e-13)


def test_one_dominant_key_selects_its_value_row():
    n, dk, dv, star = 20, 4, 6, 13
    K = np.zeros((1, 1, n, dk), np.float32)
    q = np.zeros((1, 1, dk), np.float32)
    q[0, 0, 2] = 1.0
    K[0, 0, star, 2] = 60.0
    V = rnd((1, 1, n, dv), 15)
    out = oracle.decode(q, K, V, 1.0)
    assert np.array_equal(out[0, 0], V[0, 0, star])     # deviation <= n*e^-60, below fp32
    # and with a negative scale the dominant key gets weight ~0 instead
    out2 = oracle.decode(q, K, V, -1.0)
    rest = np.delete(V[0, 0].astype(np.float64), star, axis=0).mean(axis=0)
    assert np.allclose(out2[0, 0], rest, rtol=0, atol=1e-7)


def test_two_key_closed_form_sigmoid():
    # n = 2: a[0] = sigmoid(s0 - s1) -- pins the sign of the exponent and the scale
    q = np.array([[[0.5, -1.5, 2.0]]], np.float32)
    K = np.array([[[[1.0, 0.25, -0.5], [-2.0, 1.0, 0.75]]]], np.float32)
    V = np.array([[[[1.0, 10.0], [3.0, -4.0]]]], np.float32)
    scale = 0.3
    s = scale * (K[0, 0].astype(np.float64) @ q[0, 0].astype(np.float64))
    a0 = 1.0 / (1.0 + math.exp(-(s[0] - s[1])))
    want = a0 * V[0, 0, 0] + (1 - a0) * V[0, 0, 1]
    assert np.allclose(oracle.decode(q, K, V, scale)[0, 0], want, rtol=0, atol=1e-6)


# --------------------------------------------------------------------------------------
# brute force (non-square shapes so a transposed operand or swapped d_k/d_v fails)
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("B,hq,hkv,n,dk,dv", [(1, 1, 1, 7, 3, 5), (2, 4, 2, 9, 5, 2),
                                               (1, 6, 1, 4, 2, 3), (2, 3, 3, 11, 4, 6)])
def test_oracle_f64_matches_decimal_brute_force(B, hq, hkv, n, dk, dv):
    q, K, V = rnd((B, hq, dk), 20), rnd((B, hkv, n, dk), 21), rnd((B, hkv, n, dv), 22)
    scale = 0.61
    want = brute(q, K, V, scale)
    got64 = oracle.decode_f64(q, K, V, scale)
    assert np.max(np.abs(got64 - want) / np.maximum(1e-30, np.abs(want))) < 1e-12
    got32 = oracle.decode(q, K, V, scale)
    assert np.array_equal(got32, want.astype(np.float32)) or \
        np.max(np.abs(got32 - want)) < 1e-7


def test_large_magnitude_scores_stay_finite_and_match_brute_force():
    B, hq, hkv, n, dk, dv = 1, 2, 1, 12, 6, 4
    q, K, V = 30 * rnd((B, hq, dk), 23), 30 * rnd((B, hkv, n, dk), 24), rnd((B, hkv, n, dv), 25)
    scale = 1.0                                   # scores of order 10^3..10^4
    got = oracle.decode_f64(q, K, V, scale)
    assert np.all(np.isfinite(got))
    want = brute(q, K, V, scale)
    assert np.max(np.abs(got - want)) < 1e-12


# --------------------------------------------------------------------------------------
# GQA / MQA
# --------------------------------------------------------------------------------------
def test_group_mapping_examples(golden):
    g = golden("gqa_mapping.txt")
    for key, hq, hkv in (("map_4_2", 4, 2), ("map_8_2", 8, 2)):
        want = [int(x) for x in g[key][0]]
        n, dk, dv = 3, 2, 2
        q = rnd((1, hq, dk), 30)
        K, V = rnd((1, hkv, n, dk), 31), rnd((1, hkv, n, dv), 32)
        out = oracle.decode(q, K, V, 0.7)
        for head, slab in enumerate(want):
            alone = oracle.decode(q[:, head:head + 1], K[:, slab:slab + 1],
                                  V[:, slab:slab + 1], 0.7)
            assert np.array_equal(out[0, head], alone[0, 0])
            assert slab == (head * hkv) // hq


@pytest.mark.parametrize("hkv", [8, 4, 2, 1])
def test_gqa_equals_mha_on_replicated_kv(hkv):
    hq, n, d = 8, 64, 32                           # the paper's GQA verification shapes
    q, K, V = rnd((2, hq, d), 33), rnd((2, hkv, n, d), 34), rnd((2, hkv, n, d), 35)
    scale = 1 / math.sqrt(d)
    g = hq // hkv
    a = oracle.decode(q, K, V, scale)
    b = oracle.decode(q, np.repeat(K, g, axis=1), np.repeat(V, g, axis=1), scale)
    assert np.array_equal(a, b)


def test_batch_items_are_independent():
    q, K, V = rnd((3, 4, 8), 36), rnd((3, 2, 10, 8), 37), rnd((3, 2, 10, 5), 38)
    full = oracle.decode(q, K, V, 0.3)
    for b in range(3):
        assert np.array_equal(full[b:b + 1], oracle.decode(q[b:b + 1], K[b:b + 1], V[b:b + 1], 0.3))


# --------------------------------------------------------------------------------------
# library routine: PyTorch CPU scaled_dot_product_attention
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("n", [4, 64, 256, 1024, 4096])
def test_matches_torch_sdpa_double(n):
    d = 64                                          # the paper's decode verification shapes
    q, K, V = rnd((1, 1, d), 40 + n), rnd((1, 1, n, d), 41 + n), rnd((1, 1, n, d), 42 + n)
    scale = 1 / math.sqrt(d)
    ref = F.scaled_dot_product_attention(torch.from_numpy(q).double().unsqueeze(2),
                                         torch.from_numpy(K).double(), torch.from_numpy(V).double(),
                                         scale=scale).squeeze(2).numpy()
    got = oracle.decode(q, K, V, scale)
    assert np.max(np.abs(got - ref)) < 1e-7
    # the single-precision variant sits in the paper's fp32 error band
    got32 = oracle.decode_f32(q, K, V, scale)
    assert np.max(np.abs(got32 - ref)) < 2e-6


def test_gqa_matches_torch_sdpa_per_head():
    B, hq, hkv, n, dk, dv = 2, 8, 2, 33, 16, 24
    q, K, V = rnd((B, hq, dk), 50), rnd((B, hkv, n, dk), 51), rnd((B, hkv, n, dv), 52)
    scale = 0.21
    g = hq // hkv
    Kx = torch.from_numpy(K).double().repeat_interleave(g, dim=1)
    Vx = torch.from_numpy(V).double().repeat_interleave(g, dim=1)
    ref = F.scaled_dot_product_attention(torch.from_numpy(q).double().unsqueeze(2), Kx, Vx,
                                         scale=scale).squeeze(2).numpy()
    assert np.max(np.abs(oracle.decode(q, K, V, scale) - ref)) < 1e-7
    assert np.max(np.abs(oracle.decode_f32(q, K, V, scale) - ref)) < 2e-6


# --------------------------------------------------------------------------------------
# ragged lengths, append, multi-step
# --------------------------------------------------------------------------------------
def test_varlen_equals_dense_on_prefix():
    B, hq, hkv, n_max, dk, dv = 3, 4, 2, 20, 8, 6
    q, K, V = rnd((B, hq, dk), 60), rnd((B, hkv, n_max, dk), 61), rnd((B, hkv, n_max, dv), 62)
    lens = np.array([1, 20, 7], np.int32)
    out = oracle.decode_varlen(q, K, V, lens, 0.5)
    for b in range(B):
        L = int(lens[b])
        want = oracle.decode(q[b:b + 1], K[b:b + 1, :, :L].copy(), V[b:b + 1, :, :L].copy(), 0.5)
        assert np.array_equal(out[b:b + 1], want)
    with pytest.raises(ValueError):
        oracle.decode_varlen(q, K, V, np.array([0, 1, 1], np.int32), 0.5)
    with pytest.raises(ValueError):
        oracle.decode_varlen(q, K, V, np.array([1, 21, 1], np.int32), 0.5)


def test_append_worked_example_offsets(golden):
    g = golden("append_example.txt")
    t, dk = int(g["t"][0][0]), int(g["d_k"][0][0])
    K = np.arange(100, 100 + 3 * dk, dtype=np.float32).reshape(1, 1, 3, dk)
    V = np.zeros((1, 1, 3, 1), np.float32)
    before = K.copy()
    k_new = np.array([[[7.0, 8.0, 9.0]]], np.float32)
    oracle.kv_append(K, V, k_new, np.ones((1, 1, 1), np.float32), np.array([t], np.int32))
    flat = K.reshape(-1)
    new = [int(x) for x in g["new_row_flat_offsets"][0]]
    old = [int(x) for x in g["untouched_flat_offsets"][0]]
    assert list(flat[new]) == [7.0, 8.0, 9.0]
    assert np.array_equal(flat[old], before.reshape(-1)[old])
    assert V[0, 0, t, 0] == 1.0 and V[0, 0, 0, 0] == 0.0
    # row-major offsets of a <3,2> array: l*2 + j
    gam = [int(x) for x in g["gamma_3x2"][0]]
    a = np.arange(6).reshape(3, 2)
    assert [int(a[l, j]) for l in range(3) for j in range(2)] == gam


def test_append_is_a_raw_bit_copy_and_touches_nothing_else():
    B, hkv, n_max, dk, dv = 3, 2, 5, 4, 3
    K, V = rnd((B, hkv, n_max, dk), 70), rnd((B, hkv, n_max, dv), 71)
    K0, V0 = K.copy(), V.copy()
    k_new, v_new = rnd((B, hkv, dk), 72), rnd((B, hkv, dv), 73)
    kb, vb = k_new.view(np.uint32), v_new.view(np.uint32)
    kb[0, 0, 0] = 0x80000000          # -0.0
    kb[1, 1, 2] = 0x7FC12345          # NaN with a payload
    vb[2, 0, 1] = 0xFF800000          # -inf
    vb[0, 1, 0] = 0x00000001          # smallest denormal
    pos = np.array([4, 0, 2], np.int32)
    oracle.kv_append(K, V, k_new, v_new, pos)
    for b in range(B):
        for h in range(hkv):
            assert np.array_equal(K[b, h, pos[b]].view(np.uint32), kb[b, h])
            assert np.array_equal(V[b, h, pos[b]].view(np.uint32), vb[b, h])
    mask = np.ones((B, hkv, n_max), bool)
    for b in range(B):
        mask[b, :, pos[b]] = False
    assert np.array_equal(K.view(np.uint32)[mask], K0.view(np.uint32)[mask])
    assert np.array_equal(V.view(np.uint32)[mask], V0.view(np.uint32)[mask])
    with pytest.raises(ValueError):
        oracle.kv_append(K, V, k_new, v_new, np.array([5, 0, 0], np.int32))
    with pytest.raises(ValueError):
        oracle.kv_append(K, V, k_new, v_new, np.array([0, -1, 0], np.int32))


@pytest.mark.parametrize("T,d", [(4, 8), (16, 64), (64, 64)])   # the paper's multi-step shapes
def test_multistep_equals_recompute_and_causal_attention(T, d):
    hq, hkv = 2, 1
    keys, vals, qs = rnd((T, hkv, d), 80), rnd((T, hkv, d), 81), rnd((T, hq, d), 82)
    scale = 1 / math.sqrt(d)
    K = np.zeros((1, hkv, T, d), np.float32)
    V = np.zeros((1, hkv, T, d), np.float32)
    outs = np.empty((T, hq, d), np.float32)
    for t in range(T):
        oracle.kv_append(K, V, keys[t][None], vals[t][None], np.array([t], np.int32))
        outs[t] = oracle.decode_varlen(qs[t][None], K, V, np.array([t + 1], np.int32), scale)[0]
        # (i) equals a fresh dense decode over a cache rebuilt by concatenation
        Kc = np.ascontiguousarray(keys[:t + 1].transpose(1, 0, 2))[None]
        Vc = np.ascontiguousarray(vals[:t + 1].transpose(1, 0, 2))[None]
        assert np.array_equal(outs[t], oracle.decode(qs[t][None], Kc, Vc, scale)[0])
    # (ii) equals row t of causal attention over the whole sequence
    Q = torch.from_numpy(qs).double().permute(1, 0, 2)[None]              # [1,hq,T,d]
    Kt = torch.from_numpy(keys).double().permute(1, 0, 2)[None].repeat_interleave(hq, 1)
    Vt = torch.from_numpy(vals).double().permute(1, 0, 2)[None].repeat_interleave(hq, 1)
    ref = F.scaled_dot_product_attention(Q, Kt, Vt, is_causal=True, scale=scale)[0]
    ref = ref.permute(1, 0, 2).numpy()
    assert np.max(np.abs(outs - ref)) < 1e-7


# --------------------------------------------------------------------------------------
# split-and-merge algebra used by any split-KV implementation: pinned here in double,
# before a kernel relies on it
# --------------------------------------------------------------------------------------
def test_chunk_partials_merge_to_unsplit_result():
    n, dk, dv = 53, 6, 5
    q, K, V = (rnd((dk,), 90).astype(np.float64), rnd((n, dk), 91).astype(np.float64) * 4,
               rnd((n, dv), 92).astype(np.float64))
    scale = 0.9
    want = oracle.decode_f64(q[None, None], K[None, None], V[None, None], scale)[0, 0]
    cuts = [0, 0, 5, 5, 6, 30, 53, 53]                 # includes empty chunks
    parts = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        s = scale * (K[a:b] @ q)
        if b == a:
            parts.append((-np.inf, 0.0, np.zeros(dv)))
            continue
        m = s.max()
        p = np.exp(s - m)
        parts.append((m, p.sum(), p @ V[a:b]))
    M = max(m for m, _, _ in parts)
    L = sum(l * (math.exp(m - M) if l > 0 else 0.0) for m, l, _ in parts)
    O = sum(o * (math.exp(m - M) if l > 0 else 0.0) for m, l, o in parts)
    assert np.max(np.abs(O / L - want)) < 1e-13


# --------------------------------------------------------------------------------------
# argument checking
# --------------------------------------------------------------------------------------
def test_invalid_arguments_are_rejected():
    q, K, V = rnd((1, 3, 4), 95), rnd((1, 2, 5, 4), 96), rnd((1, 2, 5, 4), 97)
    with pytest.raises(ValueError):
        oracle.decode(q, K, V, 1.0)                     # 3 % 2 != 0

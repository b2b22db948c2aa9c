"""Sequence split through the C ABI on one GPU: the row ranges that several ranks would
hold are processed one after the other (moa_decode_attn_partial), the triples are laid out
as an all-gather would leave them, and moa_combine_partials must reproduce the oracle's
result over the whole sequence.  (The exchange itself is covered on CPU by the gloo test.)"""
import numpy as np
import pytest

import moa_inputs as mi
import oracle
import paper_2607_19456_b200 as moa
from paper_2607_19456_b200 import shard
from gpu_util import TOL, max_err

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def split_decode(w, world, path=moa.PATH_AUTO):
    q, K, V = w.q(), w.K(), w.V()
    dq = torch.from_numpy(q).cuda()
    parts = torch.full((world, w.batch, w.h_q, w.d_v + 4), float("nan"), device="cuda")
    paths = set()
    moa.moa_set_option(moa.OPT_FORCE_PATH, path)
    try:
        for r in range(world):
            s, c = shard.shard_rows(w.n, world, r)
            if c == 0:
                parts[r] = shard.empty_partial(w.batch, w.h_q, w.d_v, like=dq)
                continue
            Kr = torch.from_numpy(np.ascontiguousarray(K[:, :, s:s + c])).cuda()
            Vr = torch.from_numpy(np.ascontiguousarray(V[:, :, s:s + c])).cuda()
            moa.moa_decode_attn_partial(dq, Kr, Vr, parts[r], w.batch, w.h_q, w.h_kv, c, w.d_k, w.d_v, w.scale)
            paths.add(moa.moa_last_path())
    finally:
        moa.moa_set_option(moa.OPT_FORCE_PATH, 0)
    out = torch.full((w.batch, w.h_q, w.d_v), float("nan"), device="cuda")
    moa.moa_combine_partials(parts, world, out, w.batch, w.h_q, w.d_v)
    torch.cuda.synchronize()
    assert moa.moa_device_status() == 0
    return out.cpu().numpy(), oracle.decode(q, K, V, w.scale), paths


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("hq,hkv,d,want", [(8, 2, 128, moa.PATH_STREAM), (16, 2, 128, moa.PATH_MMA),
                                           (32, 2, 64, moa.PATH_MMA), (4, 4, 32, moa.PATH_STREAM)])
def test_row_ranges_merge_to_the_unsplit_result(world, hq, hkv, d, want):
    w = mi.Workload("ss", 3000 + world + hq, 2, hq, hkv, 3001, d, d)
    got, ref, paths = split_decode(w, world)
    assert paths == {want}
    assert max_err(got, ref) <= TOL


def test_tensor_core_and_generic_kernels_export_triples_too():
    w = mi.Workload("ss", 3100, 1, 64, 1, 2500, 128, 128)
    got, ref, paths = split_decode(w, 2)
    assert paths == {moa.PATH_GROUPED} and max_err(got, ref) <= TOL
    w = mi.Workload("ss", 3101, 2, 6, 3, 77, 40, 24)
    got, ref, paths = split_decode(w, 3)
    assert paths == {moa.PATH_GENERIC} and max_err(got, ref) <= TOL


def test_more_ranks_than_row_blocks_leaves_empty_ranges():
    w = mi.Workload("ss", 3102, 2, 8, 2, 20, 128, 128)      # 20 rows over 4 ranks: 16 + 4 + 0 + 0
    got, ref, _ = split_decode(w, 4)
    assert max_err(got, ref) <= TOL


def test_one_part_equals_the_plain_call_bit_for_bit_up_to_the_division():
    w = mi.Workload("ss", 3103, 2, 8, 2, 1000, 128, 128)
    got, ref, _ = split_decode(w, 1)
    q, K, V = (torch.from_numpy(x).cuda() for x in (w.q(), w.K(), w.V()))
    out = torch.empty((w.batch, w.h_q, w.d_v), device="cuda")
    moa.moa_decode_attn(q, K, V, out, w.batch, w.h_q, w.h_kv, w.n, w.d_k, w.d_v, w.scale)
    assert float(np.max(np.abs(got - out.cpu().numpy()))) <= 2.5e-7

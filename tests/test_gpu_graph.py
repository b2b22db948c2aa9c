"""The fused decode step inside a CUDA graph: several moa_decode_step calls are captured
once (each appends its token, attends, and advances the lengths on the device) and replayed
from a restored cache; the replay must give what the oracle gives token by token."""
import numpy as np
import pytest

import moa_inputs as mi
import oracle
import paper_2607_19456_b200 as moa
from gpu_util import TOL, max_err

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.mark.parametrize("hq,hkv,d,want", [(8, 2, 128, moa.PATH_STREAM), (16, 2, 128, moa.PATH_MMA), (8, 1, 64, moa.PATH_MMA),
                                           (64, 1, 128, moa.PATH_GROUPED), (40, 1, 128, moa.PATH_GROUPED),
                                           (32, 1, 64, moa.PATH_GROUPED),      # rows of 64 features, two at a time
                                           (38, 2, 64, moa.PATH_GROUPED)])     # 19 heads per K/V head, padded lanes
def test_captured_steps_replay(hq, hkv, d, want):
    T, B, n_max = 6, 3, 400
    w = mi.Workload("gr", 5200 + hq + d, B, hq, hkv, n_max, d, d, steps=T, len_lo=1, len_hi=300)
    lens0 = w.start_lens()
    K0, V0 = w.K(), w.V()
    dK0, dV0, dl0 = torch.from_numpy(K0).cuda(), torch.from_numpy(V0).cuda(), torch.from_numpy(lens0).cuda()
    dK, dV, dl = dK0.clone(), dV0.clone(), dl0.clone()
    qs = torch.from_numpy(np.stack([w.q_step(t) for t in range(T)])).cuda()
    ks = torch.from_numpy(np.stack([w.k_new(t) for t in range(T)])).cuda()
    vs = torch.from_numpy(np.stack([w.v_new(t) for t in range(T)])).cuda()
    outs = torch.zeros((T, B, hq, d), device="cuda")
    nbytes = moa.moa_workspace_bytes(B, hq, hkv, n_max, d, d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")

    def steps():
        for t in range(T):
            moa.moa_decode_step(qs[t], dK, dV, ks[t], vs[t], outs[t], dl, B, hq, hkv, n_max, d, d, w.scale, ws, nbytes)

    steps()                                   # warm-up outside the capture (one-time set-up of the library)
    torch.cuda.synchronize()
    assert moa.moa_last_path() == want
    dK.copy_(dK0); dV.copy_(dV0); dl.copy_(dl0)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        steps()
    for _ in range(2):                        # replay twice from the restored state
        dK.copy_(dK0); dV.copy_(dV0); dl.copy_(dl0); outs.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert moa.moa_device_status() == 0
        K, V, lens = K0.copy(), V0.copy(), lens0.copy()
        got = outs.cpu().numpy()
        for t in range(T):
            oracle.kv_append(K, V, w.k_new(t), w.v_new(t), lens)
            lens = lens + 1
            assert max_err(got[t], oracle.decode_varlen(w.q_step(t), K, V, lens, w.scale)) <= TOL, t
        assert np.array_equal(dl.cpu().numpy(), lens)
        assert np.array_equal(dK.cpu().numpy().view(np.uint32), K.view(np.uint32))
        assert np.array_equal(dV.cpu().numpy().view(np.uint32), V.view(np.uint32))

"""The seeded input generator: determinism, addressing of sub-ranges, distributions."""
import numpy as np

import moa_inputs as mi


def test_same_seed_same_bits_and_different_streams_differ():
    a = mi.normal(11, mi.TID_K, (3, 5, 7))
    b = mi.normal(11, mi.TID_K, (3, 5, 7))
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    assert not np.array_equal(a, mi.normal(12, mi.TID_K, (3, 5, 7)))
    assert not np.array_equal(a, mi.normal(11, mi.TID_V, (3, 5, 7)))


def test_any_subrange_can_be_regenerated_alone():
    full = mi.normal(5, 2, (5000,))
    for start, cnt in ((0, 1), (1, 2), (301, 500), (4999, 1), (1234, 3001)):
        assert np.array_equal(full[start:start + cnt], mi.normal(5, 2, (cnt,), start=start))
    fullu = mi.uniform(5, 3, (777,))
    assert np.array_equal(fullu[100:300], mi.uniform(5, 3, (200,), start=100))


def test_chunked_threaded_fill_equals_single_shot(monkeypatch):
    a = mi.normal(3, 1, (100_003,))
    monkeypatch.setattr(mi, "_CHUNK", 4099)
    b = mi.normal(3, 1, (100_003,))
    assert np.array_equal(a, b)
    buf = np.zeros(100_003, np.float32)
    mi.normal(3, 1, (100_003,), out=buf)
    assert np.array_equal(a, buf)


def test_distributions():
    z = mi.normal(1, 1, (1 << 20,)).astype(np.float64)
    assert abs(z.mean()) < 5e-3 and abs(z.std() - 1) < 5e-3
    assert abs((z ** 3).mean()) < 2e-2 and abs((z ** 4).mean() - 3) < 5e-2
    assert abs(np.corrcoef(z[0::2], z[1::2])[0, 1]) < 5e-3
    u = mi.uniform(1, 1, (1 << 20,)).astype(np.float64)
    assert -1 < u.min() and u.max() < 1
    assert abs(u.mean()) < 5e-3 and abs(u.var() - 1 / 3) < 5e-3
    k = mi.integers(1, 6, 100_000, 512, 2048)
    assert k.min() == 512 and k.max() == 2048 and abs(k.mean() - 1280) < 10


def test_workload_table_and_slabs():
    w = mi.small_like(mi.WORKLOADS["mqa_long"], batch=2, n=300)
    K, V = w.K(), w.V()
    assert K.shape == (2, 1, 300, 128) and V.dtype == np.float32
    assert np.array_equal(w.K_slab(1, 0, rows=17), K[1, 0, :17])
    assert np.array_equal(w.V_slab(1, 0), V[1, 0])
    assert np.abs(V).max() < 1                       # U(-1,1) for this workload
    ms = mi.WORKLOADS["multi_step"]
    lens = ms.start_lens()
    assert lens.shape == (32,) and lens.min() >= 512 and lens.max() <= 2048
    assert lens.max() + ms.steps <= ms.n             # capacity holds every append
    assert ms.k_new(3).shape == (32, 8, 128) and not np.array_equal(ms.k_new(3), ms.k_new(4))
    names = list(mi.WORKLOADS)
    assert names == ["single_head", "mha", "gqa", "mqa_long", "multi_step"]

"""The analytic DRAM-traffic model (Propositions 1 and 2) against the paper's printed
tables.  The oracle's model is pinned here; the CUDA library's own `moa_min_bytes`
(host-only code, no GPU needed) is checked against the same printed values in
test_library_abi.py."""
import oracle


def mb(x):
    return x / 1e6


def close(printed, exact_mb):
    return abs(float(printed) - exact_mb) <= 0.005 + 1e-9


def test_table2_single_head(golden):
    for n, moa, sq in golden("traffic_tables.txt")["table2"]:
        n = int(n)
        assert close(moa, mb(oracle.min_bytes(1, 1, 1, n, 64, 64)))
        assert close(sq, mb(n * n * 4))
    assert oracle.min_bytes(1, 1, 1, 1024, 64, 64) == (64 + 1024 * 64 + 1024 * 64 + 64) * 4


def test_table4_multi_step(golden):
    d = 64
    for T, app, dec, sq in golden("traffic_tables.txt")["table4"]:
        T = int(T)
        assert close(app, mb(T * (d + d) * 4))                      # Proposition 2, T times
        assert close(dec, mb(sum(oracle.min_bytes(1, 1, 1, t, d, d) for t in range(1, T + 1))))
        assert close(sq, mb(sum(t * t * 4 for t in range(1, T + 1))))


def test_table6_gqa(golden):
    n, d, hq = 1024, 64, 32
    for hkv, kv, total in golden("traffic_tables.txt")["table6"]:
        hkv = int(hkv)
        tot = oracle.min_bytes(1, hq, hkv, n, d, d)
        assert close(total, mb(tot))
        assert close(kv, mb(tot - hq * (d + d) * 4))
        assert tot - hq * (d + d) * 4 == hkv * n * (d + d) * 4


def test_model_is_linear_in_batch_and_uses_dk_plus_dv():
    assert oracle.min_bytes(3, 8, 2, 100, 16, 48) == 3 * (2 * 100 * 64 + 8 * 64) * 4
    # exceeds 32 bits without overflow
    assert oracle.min_bytes(16, 32, 8, 8192, 128, 128) == 1074266112
    assert oracle.min_bytes(64, 64, 64, 1 << 20, 128, 128) == 64 * (64 * (1 << 20) * 256 + 64 * 256) * 4

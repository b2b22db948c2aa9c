"""Host-side checks of the CUDA library that need no GPU: it loads, exports every symbol
the public header declares, validates arguments before touching CUDA, and its byte model
reproduces the paper's printed traffic tables."""
import os
import re

import pytest

import paper_2607_19456_b200 as moa
from paper_2607_19456_b200 import build as moa_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    moa_build.build()            # cross-compiles with nvcc; no GPU needed
    return moa.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "moa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moa_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert {"moa_decode_attn", "moa_decode_attn_varlen", "moa_kv_append", "moa_workspace_bytes",
            "moa_device_status", "moa_min_bytes", "moa_strerror"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_binding_has_the_same_names(L):
    for n in declared_functions():
        assert callable(getattr(moa, n)), n


def test_arguments_are_validated_before_any_cuda_call(L):
    # On a machine without a GPU these return the argument error, not MOA_ERR_CUDA.
    assert L.moa_decode_attn(None, 16, 16, 16, 1, 1, 1, 1, 64, 64, 1.0, None) == moa.ERR_INVALID
    assert L.moa_decode_attn(16, 16, 16, 16, 1, 3, 2, 1, 64, 64, 1.0, None) == moa.ERR_INVALID
    assert L.moa_decode_attn(16, 16, 16, 16, 0, 1, 1, 1, 64, 64, 1.0, None) == moa.ERR_INVALID
    assert L.moa_decode_attn(16, 16, 16, 16, 1, 1, 1, 0, 64, 64, 1.0, None) == moa.ERR_INVALID
    assert L.moa_decode_attn(16, 16, 16, 16, 1, 1, 1, 1, 64, 64, float("inf"), None) == moa.ERR_INVALID
    assert L.moa_decode_attn(16, 16, 16, 16, 1, 1, 1, 1, 4096, 64, 1.0, None) == moa.ERR_UNSUPPORTED
    assert L.moa_decode_attn(18, 16, 16, 16, 1, 1, 1, 1, 64, 64, 1.0, None) == moa.ERR_ALIGN
    assert L.moa_kv_append(None, 16, 16, 16, 16, 1, 1, 1, 1, 1, None) == moa.ERR_INVALID
    assert L.moa_kv_append(16, 16, 16, 16, 16, 1, 1, 0, 1, 1, None) == moa.ERR_INVALID
    assert L.moa_kv_append(16, 16, 16, 16, 17, 1, 1, 1, 1, 1, None) == moa.ERR_ALIGN
    assert L.moa_lens_add(None, 1, 1, None) == moa.ERR_INVALID
    assert L.moa_decode_step(16, 16, 16, 16, 16, 16, None, 1, 1, 1, 1, 64, 64, 1.0, None, 0, None) == moa.ERR_INVALID
    assert L.moa_decode_attn_host(None, 16, 16, 16, 1, 1, 1, 1, 64, 64, 1.0) == moa.ERR_INVALID
    assert L.moa_device_status(None, None) == moa.ERR_INVALID
    assert L.moa_set_option(99, 0) == moa.ERR_INVALID
    assert L.moa_set_option(moa.OPT_FORCE_PATH, 7) == moa.ERR_INVALID
    assert moa.moa_workspace_bytes(1, 3, 2, 10, 64, 64) == 0
    with pytest.raises(moa.MoaError) as e:
        moa.moa_decode_attn(None, 16, 16, 16, 1, 1, 1, 1, 64, 64, 1.0, stream=0)
    assert e.value.code == moa.ERR_INVALID and "invalid argument" in str(e.value)


def test_no_cpu_fallback_without_a_gpu(L):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    # valid arguments, no device: the call must fail loudly instead of computing on the CPU
    assert L.moa_decode_attn(16, 16, 16, 16, 1, 1, 1, 1, 64, 64, 1.0, None) == moa.ERR_CUDA


def test_strerror_covers_every_code():
    texts = {moa.strerror(c) for c in range(7)}
    assert len(texts) == 7 and "unknown" in moa.strerror(99)


def test_library_byte_model_matches_the_printed_tables(golden):
    g = golden("traffic_tables.txt")

    def close(printed, nbytes):
        return abs(float(printed) - nbytes / 1e6) <= 0.005 + 1e-9

    for n, mb, _ in g["table2"]:
        assert close(mb, moa.moa_min_bytes(1, 1, 1, int(n), 64, 64))
    for T, _, dec, _ in g["table4"]:
        assert close(dec, sum(moa.moa_min_bytes(1, 1, 1, t, 64, 64) for t in range(1, int(T) + 1)))
    for hkv, _, total in g["table6"]:
        assert close(total, moa.moa_min_bytes(1, 32, int(hkv), 1024, 64, 64))
    assert moa.moa_min_bytes(4, 64, 1, 131072, 128, 128) == 537133056


def test_product_code_never_touches_the_oracle():
    # the library, its binding and the input generator must not import or link the oracle
    pkg = os.path.join(ROOT, "paper_2607_19456_b200")
    files = [os.path.join(dp, f) for dp, _, fs in os.walk(pkg) for f in fs
             if f.endswith((".py", ".cu", ".cuh", ".h"))] + [os.path.join(ROOT, "moa_inputs.py"),
                                                             os.path.join(ROOT, "include", "moa.h")]
    pat = re.compile(r"import\s+oracle|from\s+oracle|moa_oracle|oracle/")
    for f in files:
        assert not pat.search(open(f).read()), f

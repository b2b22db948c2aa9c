"""Failure detection inside a kernel, without faulting the GPU: every wait in the library is
bounded, and when one runs out the kernel reports it and returns.  Here the wait is made to
run out on purpose on the smallest case: one CTA of the FMA streaming kernel, a wait limit of
a few thousand polls, and one row block whose copies are announced but never issued (nothing
is in flight and nothing is out of bounds)."""
import numpy as np
import pytest

import moa_inputs as mi
import oracle
import paper_2607_19456_b200 as moa
from gpu_util import TOL, Guarded, max_err

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def test_an_expired_wait_is_reported_and_the_library_stays_usable():
    w = mi.Workload("we", 6100, 1, 1, 1, 256, 64, 64)               # one unit, one CTA
    q, K, V = w.q(), w.K(), w.V()
    gq, gK, gV = Guarded(q), Guarded(K), Guarded(V)
    gout = Guarded(shape=(1, 1, 64), fill=-7.0)
    args = (gq.ptr, gK.ptr, gV.ptr, gout.ptr, 1, 1, 1, w.n, 64, 64, w.scale)
    moa.moa_set_option(moa.OPT_WAIT_LIMIT, 2000)
    moa.moa_set_option(moa.OPT_TEST_SKIP_COPY, 5)                   # row block 5 of 16 never arrives
    try:
        moa.moa_decode_attn(*args)                                  # returns: the wait gives up
        torch.cuda.synchronize()
        assert moa.moa_last_path() == moa.PATH_STREAM
        assert moa.moa_device_status() & moa.STATUS_WAIT_TIMEOUT
    finally:
        moa.moa_set_option(moa.OPT_TEST_SKIP_COPY, -1)
        moa.moa_set_option(moa.OPT_WAIT_LIMIT, 0)
    for g in (gq, gK, gV, gout):
        assert g.guards_intact()
    assert moa.moa_device_status() == 0                             # reading the status cleared it
    moa.moa_decode_attn(*args)                                      # the next ordinary call is correct
    torch.cuda.synchronize()
    assert moa.moa_device_status() == 0
    assert max_err(gout.host(), oracle.decode(q, K, V, w.scale)) <= TOL

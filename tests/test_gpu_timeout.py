"""The time-out path on a GPU, in its one safe form: a one-warp kernel whose bounded wait (the kernels' own
wait routine) expires after a millisecond and which then returns normally.  Nothing hangs or faults: the status
word is set, read once, and the library keeps working."""
import numpy as np
import pytest

import oracle
import paper_2609_36800_b200 as bd
from paper_2609_36800_b200 import synth

from gpu_util import assert_parity, run_gemm

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_once_and_the_library_stays_usable():
    assert bd.last_device_status() == (0, 0)
    bd.selftest_timeout(limit_cycles=1_000_000, site=77)          # ~0.5 ms
    assert bd.last_device_status() == (bd.STATUS_TIMEOUT, 77)
    assert "wait" in bd.status_string(bd.STATUS_TIMEOUT)
    assert bd.last_device_status() == (0, 0)                       # cleared by the query
    # the first expiry wins, the second is not recorded over it
    bd.selftest_timeout(limit_cycles=200_000, site=5)
    bd.selftest_timeout(limit_cycles=200_000, site=6)
    assert bd.last_device_status() == (bd.STATUS_TIMEOUT, 5)
    # a product after it matches the oracle (decode and tiled schedules)
    for shape in [(3, 2, 384, 512), (2, 48, 256, 384)]:
        wl = synth.Workload("t", B=shape[0], m=shape[1], N=shape[2], K=shape[3], seed=17)
        X, W, bits, alpha = synth.make_inputs(wl)
        assert_parity(run_gemm(X, W, bits, alpha), oracle.gemm(X, W, bits, alpha), str(shape))


def test_selftest_refuses_limits_that_would_not_end_soon():
    with pytest.raises(bd.BitDeltaError):
        bd.selftest_timeout(limit_cycles=10**12)
    with pytest.raises(bd.BitDeltaError):
        bd.selftest_timeout(limit_cycles=10)

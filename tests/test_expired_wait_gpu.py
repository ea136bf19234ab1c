"""The bounded device-side waits: one that is made to run out (a barrier nothing completes, with a limit of a
million cycles) is reported as MOA_ERR_TIMEOUT, once, and the device stays usable.  Nothing here faults or hangs."""
import math
import time

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

import oracle
from paper_2609_33916_b200 import inputs as mi


def test_expired_wait_is_reported_once_and_the_device_stays_usable():
    import gpu_harness as H
    from paper_2609_33916_b200 import binding as mb
    from paper_2609_33916_b200 import build as mbuild
    mbuild.build()
    assert mb.moa_last_device_status() == mb.MOA_OK
    t0 = time.perf_counter()
    assert mb.moa_selftest_expired_wait(1_000_000) == mb.MOA_OK           # about half a millisecond on the device
    assert mb.moa_last_device_status() == mb.MOA_ERR_TIMEOUT
    assert time.perf_counter() - t0 < 1.0                                  # it gave up after its limit, not after seconds
    assert mb.moa_last_device_status() == mb.MOA_OK                       # reported once, then cleared
    # the context is intact: a normal call gives correct results
    inp = mi.make_inputs(1, 2, 256, 128, seed=5, dtype="bf16")
    f = {k: mi.to_f64(v, "bf16") for k, v in inp.items()}
    ref = oracle.attn_fwd_bwd(f["Q"], f["K"], f["V"], f["dO"], True, 1.0 / math.sqrt(128))
    got = H.run_library(inp, "bf16", True, 1.0 / math.sqrt(128))
    H.assert_close(got, ref, H.TOL_BF16, tag="after an expired wait")
    # limits are clamped: a request for "no limit" still ends (at most about a second)
    assert mb.moa_selftest_expired_wait(50) == mb.MOA_OK
    assert mb.moa_last_device_status() == mb.MOA_ERR_TIMEOUT
    assert mb.moa_last_device_status() == mb.MOA_OK

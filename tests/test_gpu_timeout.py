"""The time-out path of the bounded waits, made to run on purpose and harmlessly: a one-CTA
kernel waits (limit 1 ms, passed as an argument) on a barrier nobody arrives at.  The kernel
must return, the error word must be reported exactly once, and the library must go on working."""
import math

import numpy as np
import pytest

import paper_2410_20926_b200 as ta
from paper_2410_20926_b200 import inputs as ta_inputs

from helpers import gpu_forward

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_once_and_the_context_stays_usable():
    import torch
    torch.cuda.synchronize()
    assert ta.ta_device_status(check=False) == ta.TA_OK
    rc, report = ta.ta_selftest_wait_timeout(1000)
    assert rc == ta.TA_OK
    expired, left_by_flag, copy_landed, waited_ns = report
    assert expired == 1            # the wait with the short limit gave up ...
    assert left_by_flag == 1       # ... the other role left through the abort flag, not its own 2 s limit
    assert copy_landed == 1        # ... and the copy in flight was waited for before leaving
    assert 1_000_000 <= waited_ns < 100_000_000
    assert ta.ta_device_status(check=False) == ta.TA_ERR_TIMEOUT
    assert ta.ta_device_status(check=False) == ta.TA_OK             # reported once, then cleared
    with pytest.raises(ta.TaError):
        ta.ta_selftest_wait_timeout(1000)
        ta.ta_device_status()
    # the next forward pass runs and is correct
    B, H, Hkv, D, dims = 1, 4, 2, 128, [8, 16, 32]
    N = math.prod(dims)
    inp = ta_inputs.make_inputs(B, H, Hkv, N, D, "bf16", 601)
    a = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16")
    b = gpu_forward(inp, B, H, Hkv, N, D, dims, True, "bf16", ta.TA_FLAG_PAIR_HOPS)
    np.testing.assert_array_equal(a, b)


def test_selftest_rejects_limits_outside_the_documented_range():
    assert ta.ta_selftest_wait_timeout(0, check=False)[0] == ta.TA_ERR_INVALID_ARG
    assert ta.ta_selftest_wait_timeout(2_000_000, check=False)[0] == ta.TA_ERR_INVALID_ARG

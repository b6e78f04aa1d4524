"""The bounded-wait path: a device-side wait that runs out is reported, nothing hangs, and the device stays usable.

Every wait of the tensor-core kernels on a shared-memory barrier has a limit in clock cycles; when it runs out the
thread block raises an abort flag, records the time-out in the device status word, frees its tensor memory and
returns.  The test makes exactly that happen in the permitted way: a one-block kernel waits, with a limit of 10^5 cycles
(about 50 microseconds), on a barrier that nothing arrives on.  No trap, no fault, no endless loop."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_1911_05181_b200 import binding as ul
from helpers import TOL, gpu_sgemm

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_device_stays_usable():
    torch.cuda.synchronize()
    assert ul.last_device_status() == ul.OK
    for limit in (100_000, 2_000_000):
        assert ul.debug_wait_timeout(limit) == ul.OK           # enqueued; returns by itself
        assert ul.last_device_status() == ul.ERR_DEVICE_TIMEOUT     # synchronises, reports, clears
        assert ul.last_device_status() == ul.OK
    # tensor memory was given back and the context is intact: a product on the tensor cores runs clean afterwards
    M, N, K = 384, 512, 256
    A, B, C = si.gemm_operands(4, M, K, K, N, M, N)
    got = gpu_sgemm("N", "N", M, N, K, 1.0, A, K, B, N, 0.0, C.copy(), N, ul.MATH_3XTF32)
    assert oracle.rel_l2(got, oracle.sgemm("N", "N", M, N, K, 1.0, A, K, B, N, 0.0)) <= TOL[ul.MATH_3XTF32]
    assert ul.last_device_status() == ul.OK


def test_limit_out_of_range_is_refused_on_the_host():
    assert ul.debug_wait_timeout(0) == ul.ERR_INVALID_ARG
    assert ul.debug_wait_timeout(3_000_000_000) == ul.ERR_INVALID_ARG

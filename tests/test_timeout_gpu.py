"""The give-up path of the tensor-core kernels' bounded barrier waits, exercised without stalling
a real launch: a one-thread kernel waits with the same helper on a barrier nothing arrives on, the
wait runs out after a millisecond, the status word carries the bit, FREQKV_ERR_TIMEOUT is reported
once, and the context goes on working.  (A wait that gives up and returns -- not a fault.)"""
import time

import pytest
import torch

from paper_2505_00570_b200 import binding as fk
from paper_2505_00570_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


def test_a_bounded_wait_runs_out_and_the_context_stays_usable():
    ctx = fk.Context(0)
    try:
        assert ctx.last_device_status() == fk.OK
        t0 = time.perf_counter()
        ctx.selftest_bounded_wait(1_000_000)          # 1 ms
        status = ctx.last_device_status()             # synchronises the stream
        elapsed = time.perf_counter() - t0
        assert status == fk.ERR_TIMEOUT
        assert "bounded wait" in ctx.last_error()
        assert elapsed < 1.0, "the wait did not give up at its limit"
        assert ctx.last_device_status() == fk.OK      # the report cleared the word
        # the same context compresses correctly afterwards, on the tensor-core path too
        w = synth.Workload("after", 1, 1, 2, 128, 700, torch.bfloat16, 4, 0.9, 2, synth.BASE_SEED + 90)
        parity.check_compress(ctx, w, 700, 348, 4, fk.GEMM)
        assert ctx.last_device_status() == fk.OK
    finally:
        ctx.close()


def test_wait_limit_arguments():
    ctx = fk.Context(0)
    try:
        ctx.set_wait_limit(50_000_000)
        for bad in (0, 999):
            with pytest.raises(fk.FreqKVError) as e:
                ctx.set_wait_limit(bad)
            assert e.value.status == fk.ERR_INVALID_ARG
        with pytest.raises(fk.FreqKVError) as e:
            ctx.selftest_bounded_wait(2_000_000_000)   # beyond the probe's own ceiling of one second
        assert e.value.status == fk.ERR_INVALID_ARG
        # a shorter limit does not disturb a healthy launch
        w = synth.Workload("short", 1, 1, 2, 128, 700, torch.bfloat16, 4, 0.9, 2, synth.BASE_SEED + 91)
        parity.check_compress(ctx, w, 700, 348, 4, fk.GEMM)
        assert ctx.last_device_status() == fk.OK
    finally:
        ctx.close()

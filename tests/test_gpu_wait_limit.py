"""Bounded device-side waits: a wait that can never be satisfied gives up, reports it through
the status word and leaves the context usable (no trap, no hang)."""

import time

import pytest
import torch

import paper_2609_32518_b200 as U
import workloads as W
from test_gpu_attn import run

pytestmark = pytest.mark.gpu


def test_wait_runs_out_status_is_reported_and_work_goes_on():
    assert U.poll_status() == 0
    t0 = time.perf_counter()
    U.selftest_wait_limit(2_000_000)            # about a millisecond of SM clock
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0
    assert U.poll_status() == -4                # UNSTEP_ERR_TIMEOUT, reported once
    assert U.poll_status() == 0
    run(W.WORKLOADS["cfg1"])                    # the library still works in the same context


def test_limit_argument_is_checked():
    with pytest.raises(U.UnstepError):
        U.selftest_wait_limit(0)
    with pytest.raises(U.UnstepError):
        U.selftest_wait_limit(5_000_000_000)


def test_shutdown_frees_scratch_and_the_library_keeps_working():
    run(W.WORKLOADS["cfg1_wrapped"])
    before = torch.cuda.mem_get_info()[0]
    U.shutdown()
    after = torch.cuda.mem_get_info()[0]
    assert after >= before                      # the scratch (tens of MB) went back to the driver
    run(W.WORKLOADS["cfg1_wrapped"])            # and is made again on demand

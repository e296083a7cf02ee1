"""The bounded device-side waits on real hardware: a wait on an mbarrier that nothing completes gives up
after its limit, the kernel returns with the status word set, and the context stays usable."""
import time

import pytest
import torch

import dvm_workloads as wl
import paper_2603_24239_b200 as dvm
from tests.parity_util import check, gpu_run, oracle_run

pytestmark = pytest.mark.gpu

DVM_ERR_DEVICE_TIMEOUT = -7


@pytest.mark.parametrize("which", [0, 1, 2])  # the interpreter's barrier wait, the matmul kernel's, the level wait
def test_wait_runs_out_and_reports(which):
    assert dvm.last_device_status() == 0
    t0 = time.perf_counter()
    dvm.selftest_bounded_wait(which)
    status = dvm.last_device_status()          # synchronises the stream
    dt = time.perf_counter() - t0
    assert status == DVM_ERR_DEVICE_TIMEOUT
    assert 1.0 < dt < 10.0, dt                 # the limit is 2 s
    assert dvm.last_device_status() == 0       # reading the status clears it
    # the context is intact: a normal program still runs and matches the oracle
    prog = wl.program_c1()
    ins = wl.inputs_c1()
    outs, _ = gpu_run(prog, ins)
    check(prog, outs, oracle_run(prog, ins))

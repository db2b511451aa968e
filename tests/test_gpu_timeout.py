"""Failure handling without a fault: a bounded device-side wait that runs out, and the call after it.

Every role of the int8 GEMM kernel waits on its barriers with a time budget; when a wait gives up it records a code in the
workspace's status word, which gemm2m_device_status() turns into GEMM2M_ERR_DEVICE_TIMEOUT.  gemm2m_debug_wait_selftest
runs that same wait, with a short budget, on a barrier that nobody arrives on (one thread, no pipeline, no bulk copy, no
TMEM), so the wait gives up by construction and the kernel returns: nothing hangs, traps or faults.
"""
import time

import pytest
import torch

from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host  # noqa: E402


def test_a_wait_that_runs_out_is_reported_once_and_the_next_call_is_clean():
    m, n, k, nmod = 300, 260, 200, 16
    A, B = inputs.complex_inputs(m, n, k, seed=41)
    dA, dB = to_dev(A), to_dev(B)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, nmod)):
        C0 = empty_dev(m, n, torch.complex128)
        b.zgemm2m(dA, dB, C0, nmod)
        b.device_status()                                   # clean
        b.debug_wait_selftest(100_000)                      # warm-up of the launch itself (module load), reported below
        with pytest.raises(b.Gemm2mError) as err:
            b.device_status()
        assert err.value.status == b.ERR_DEVICE_TIMEOUT
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        b.debug_wait_selftest(100_000)                      # 0.1 ms budget
        with pytest.raises(b.Gemm2mError) as err:
            b.device_status()                               # synchronises the stream, reads and clears the status word
        elapsed = time.perf_counter() - t0
        assert err.value.status == b.ERR_DEVICE_TIMEOUT
        assert elapsed < 0.010, elapsed                     # the wait gave up after its budget, not after the 2 s default
        b.device_status()                                   # reported once: the word is clear again
        C1 = empty_dev(m, n, torch.complex128)
        b.zgemm2m(dA, dB, C1, nmod)                         # same workspace, next ordinary call
        b.device_status()
        assert (to_host(C1) == to_host(C0)).all()


def test_selftest_needs_a_workspace():
    b.set_workspace(None)
    with pytest.raises(b.Gemm2mError) as err:
        b.debug_wait_selftest(100_000)
    assert err.value.status == b.ERR_WORKSPACE

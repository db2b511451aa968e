"""zgemm2m_host: the end-to-end entry point on host operands.  Its result must be bit for bit that of zgemm2m on device
operands (same scale factors, same planes), whatever the panel count, padding or memory kind."""
import numpy as np
import pytest
import torch

from oracle import direct, staged
from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host, ulp_distance  # noqa: E402


def host_colmajor(a, ld=None, pin=True, fill=None):
    """numpy (rows, cols) -> CPU tensor view of that shape stored column-major with leading dimension ld."""
    rows, cols = a.shape
    ld = rows if ld is None else ld
    buf = torch.empty((cols, max(ld, 1)), dtype=torch.complex128, pin_memory=pin)
    if fill is not None:
        buf.fill_(fill)
    view = buf[:, :rows].t()
    view.copy_(torch.from_numpy(np.ascontiguousarray(a)))
    return buf, view


def run_device(A, B, nmod):
    m, k = A.shape
    n = B.shape[1]
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, nmod)):
        C = empty_dev(m, n, torch.complex128)
        b.zgemm2m(to_dev(A), to_dev(B), C, nmod)
        b.device_status()
        return to_host(C)


@pytest.mark.parametrize("shape,nmod,pin", [((200, 150, 300), 16, True), ((129, 2300, 128), 14, True), ((64, 64, 64), 3, False),
                                            ((1500, 4100, 260), 16, True), ((33, 19, 50), 24, True), ((300, 1024, 200), 20, False)])
def test_host_call_is_bitwise_the_device_call(shape, nmod, pin):
    m, n, k = shape
    A, B = inputs.complex_inputs(m, n, k, seed=13, dist="phi", phi=1.0)
    want = run_device(A, B, nmod)
    _, hA = host_colmajor(A, ld=m + 3, pin=pin)
    _, hB = host_colmajor(B, ld=k + 5, pin=pin)
    bufC, hC = host_colmajor(np.zeros((m, n), dtype=np.complex128), ld=m + 2, pin=pin, fill=-7)
    hC.fill_(0)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM_HOST, m, n, k, nmod)):
        b.zgemm2m_host(hA, hB, hC, nmod)
        torch.cuda.synchronize()
        b.device_status()
        got = hC.numpy().copy()
        assert np.array_equal(got, want)
        assert (bufC[:, m:] == -7).all()                      # padding rows of C_host untouched
        # a second call on new data through the same workspace and events (the device copies are reused)
        A2, B2 = inputs.complex_inputs(m, n, k, seed=14, dist="uniform")
        hA.copy_(torch.from_numpy(np.ascontiguousarray(A2)))
        hB.copy_(torch.from_numpy(np.ascontiguousarray(B2)))
        b.zgemm2m_host(hA, hB, hC, nmod)
        b.zgemm2m_host(hA, hB, hC, nmod)                      # back to back, no host synchronisation between the calls
        torch.cuda.synchronize()
        b.device_status()
        got2 = hC.numpy().copy()
    assert np.array_equal(got2, run_device(A2, B2, nmod))
    Cref, D = direct.zgemm4m_dd(A2, B2)
    if nmod >= 16:
        assert direct.componentwise_error(got2, Cref, D) <= 1e-14


def test_host_call_orders_itself_on_the_callers_stream_and_handles_degenerate_sizes():
    m, n, k, nmod = 700, 2100, 150, 16
    A, B = inputs.complex_inputs(m, n, k, seed=3, dist="uniform")
    want = run_device(A, B, nmod)
    _, hA = host_colmajor(A)
    _, hB = host_colmajor(B)
    _, hC = host_colmajor(np.zeros((m, n), dtype=np.complex128))
    st = torch.cuda.Stream()
    with Workspace(b.workspace_bytes(b.OP_ZGEMM_HOST, m, n, k, nmod)):
        done = torch.cuda.Event()
        with torch.cuda.stream(st):
            b.zgemm2m_host(hA, hB, hC, nmod, st)
            done.record(st)
        done.synchronize()                                    # only the caller's stream is waited for
        assert np.array_equal(hC.numpy(), want)
        b.device_status()
        # k = 0: C = 0; empty m or n: no-op
        _, hA0 = host_colmajor(np.zeros((m, 0), dtype=np.complex128))
        _, hB0 = host_colmajor(np.zeros((0, n), dtype=np.complex128))
        hC.fill_(5)
        b.zgemm2m_host(hA0, hB0, hC, nmod)
        torch.cuda.synchronize()
        assert (hC.numpy() == 0).all()
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, 64, 64, 64, 16)):          # enough for zgemm2m, not for the device copies
        _, a = host_colmajor(np.ones((64, 64), dtype=np.complex128))
        _, c = host_colmajor(np.zeros((64, 64), dtype=np.complex128))
        with pytest.raises(b.Gemm2mError):
            b.zgemm2m_host(a, a, c, 16)                       # workspace without room for the device copies

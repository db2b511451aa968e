"""The allocation-free entry point against the regular one.

gemm2m_zscale_exponents_static serves callers that cannot allocate device memory (no workspace to hand over); its
scratch is an array built into the library.  This file is collected last on purpose: a run that stops at the first
failure has then already run every other test.  The checks: two calls in a row through the C-ABI give exactly the
exponents zgemm2m leaves in its workspace (integers, so the tolerance is equality), the second call is not
polluted by what the first left in the shared scratch, and oversized requests are refused.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev  # noqa: E402
from oracle import staged  # noqa: E402


def exponents_from_oracle(A, k, nmod):
    """The staged oracle's rule for the rows of A (Algorithm 1 step 2), from the budget of the first nmod moduli."""
    M = staged.product(staged.hybrid_moduli(nmod))
    _, PA, _, ck = staged.scaling_targets(M, k)
    return staged.scaling_exponents(A, 1, PA, ck)


def exponents_from_zgemm2m(A, B, nmod):
    m, k = A.shape
    n = B.shape[1]
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, nmod)) as ws:
        b.zgemm2m(to_dev(A), to_dev(B), empty_dev(m, n, torch.complex128), nmod)
        b.device_status()
        return ws.stages(b.OP_ZGEMM, m, n, k, nmod)["eA"]


def test_static_scratch_entry_point_matches_zgemm2m_on_two_calls_in_a_row():
    nmod = 16
    m, n, k = 300, 40, 500
    A1, B = inputs.complex_inputs(m, n, k, seed=31, dist="phi", phi=2.0)
    A2 = np.asfortranarray(A1[:257] * 2.0 ** -40)      # fewer rows, much smaller entries: stale maxima would show
    A2[5, :] = 0
    want1 = exponents_from_zgemm2m(A1, B, nmod)
    want2 = exponents_from_zgemm2m(A2, B, nmod)
    b.set_workspace(None)                               # nothing registered: the new call must not need it
    e1 = torch.full((m,), 12345, dtype=torch.int32, device="cuda")
    e2 = torch.full((257,), 12345, dtype=torch.int32, device="cuda")
    dA1, dA2 = to_dev(A1), to_dev(A2)
    before = torch.cuda.memory_allocated()
    b.zscale_exponents_static(dA1, e1, nmod)            # first call on this device also looks up the scratch address
    b.zscale_exponents_static(dA2, e2, nmod)            # second call right behind it, same stream
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    assert (e1.cpu().numpy() == want1).all()
    assert (e2.cpu().numpy() == want2).all()
    assert (e1.cpu().numpy() == exponents_from_oracle(A1, k, nmod)).all()      # and against the oracle itself, not only zgemm2m
    assert (e2.cpu().numpy() == exponents_from_oracle(A2, k, nmod)).all()
    assert want2[5] == 0 and (want2[:5] < want1[:5]).all()


def test_static_scratch_entry_point_refuses_oversized_and_bad_arguments():
    L = b.lib()
    one = ctypes.c_void_p(256)                          # never dereferenced: checks come before any launch
    big = b.STATIC_MAX_ROWS + 1
    assert L.gemm2m_zscale_exponents_static(big, 4, one, big, 16, one, None) == 3       # GEMM2M_ERR_WORKSPACE
    assert L.gemm2m_zscale_exponents_static(4, 4, one, 3, 16, one, None) == 1           # lda < m
    assert L.gemm2m_zscale_exponents_static(4, 4, one, 4, 0, one, None) == 2            # nmod out of range
    assert L.gemm2m_zscale_exponents_static(0, 4, None, 1, 16, None, None) == 0         # empty: nothing to do
    with pytest.raises(ValueError, match="built-in scratch"):
        A = torch.empty((4, big), dtype=torch.complex128, device="cuda").t()
        b.zscale_exponents_static(A, torch.empty(big, dtype=torch.int32, device="cuda"))

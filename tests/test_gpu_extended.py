"""GPU parity of the BLAS-style extended entry points (alpha, beta, transposed / conjugated operands) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import direct, staged
from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host, ulp_distance  # noqa: E402

TOL_Z, TOL_C = 1e-14, 2e-6


def stored(X, trans):
    """The matrix as the caller stores it so that op(stored) = X."""
    return np.asfortranarray(X if trans == "N" else (X.T if trans == "T" else X.conj().T))


def run_ex(ta, tb, alpha, A, B, beta, C0, nmod, cplx=torch.complex128, kernel=0, ldc=None):
    m, k = A.shape
    n = B.shape[1]
    op = b.OP_ZGEMM if cplx == torch.complex128 else b.OP_CGEMM
    b.debug_set_gemm_kernel(kernel)
    try:
        with Workspace(b.workspace_bytes(op, m, n, k, nmod)) as ws:
            C = empty_dev(m, n, cplx, ld=ldc, fill=-3.0)
            if C0 is not None:
                C.copy_(to_dev(C0))
            fn = b.zgemm2m_ex if op == b.OP_ZGEMM else b.cgemm2m_ex
            fn(ta, tb, alpha, to_dev(stored(A, ta)), to_dev(stored(B, tb)), beta, C, nmod)
            b.device_status()
            st = ws.stages(op, m, n, k, nmod)
            return to_host(C), st
    finally:
        b.debug_set_gemm_kernel(0)


@pytest.mark.parametrize("ta,tb", [("N", "N"), ("T", "N"), ("N", "T"), ("C", "N"), ("N", "C"), ("C", "C"), ("T", "C")])
def test_transposed_and_conjugated_operands_give_the_same_stages(ta, tb):
    """op(A) op(B) with alpha = 1, beta = 0: scale exponents, residue planes and C+- planes are those of the staged
    oracle run on the explicit op(A), op(B); the result equals the plain entry point's bit for bit."""
    m, n, k, nmod = 150, 131, 300, 16
    A, B = inputs.complex_inputs(m, n, k, seed=41, dist="phi", phi=1.0)      # A = op(A_stored), B = op(B_stored)
    C, st = run_ex(ta, tb, None, A, B, None, None, nmod, kernel=1)
    ref = staged.zgemm2m_staged(A, B, nmod)
    assert (st["eA"] == ref["eA"]).all() and (st["eB"] == ref["eB"]).all()
    for j in range(nmod):
        for sgn in range(2):
            assert (st["Apm"][sgn, j, :, :k] == ref["Apm"][j][sgn]).all(), ("Apm", sgn, j)
            assert (st["Bpm"][sgn, j, :, :k] == ref["Bpm"][j][sgn].T).all(), ("Bpm", sgn, j)
            assert (st["Cpm"][sgn, j, :, :m] == ref["Cpm"][j][sgn].T).all(), ("Cpm", sgn, j)
    assert ulp_distance(C.real, ref["C"].real).max() <= 1 and ulp_distance(C.imag, ref["C"].imag).max() <= 1
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, nmod)):
        Cp = empty_dev(m, n, torch.complex128)
        b.zgemm2m(to_dev(A), to_dev(B), Cp, nmod)
        assert (to_host(Cp) == C).all()


@pytest.mark.parametrize("alpha,beta", [(2.0, 0.0), (1.0, 1.0), (0.75 - 1.5j, -0.5 + 0.25j), (-1.0, 3.0j), (1.0, 0.0)])
@pytest.mark.parametrize("ta,tb", [("N", "N"), ("C", "T")])
def test_alpha_beta_against_the_definition(alpha, beta, ta, tb):
    m, n, k, nmod = 200, 170, 257, 16
    A, B = inputs.complex_inputs(m, n, k, seed=43)
    C0, _ = inputs.complex_inputs(m, 1, n, seed=44)                           # m x n
    C, _ = run_ex(ta, tb, alpha, A, B, beta, C0, nmod, ldc=m + 9)
    Cref, D = direct.zgemm_ex_dd("N", "N", alpha, A, B, beta, C0)
    assert direct.componentwise_error(C[:m], Cref, D) <= TOL_Z
    assert (C[m:] == -3.0).all()                                              # padding rows of C untouched


def test_beta_zero_ignores_c_and_alpha_zero_ignores_a_b():
    m, n, k, nmod = 64, 48, 96, 16
    A, B = inputs.complex_inputs(m, n, k, seed=45)
    C0, _ = inputs.complex_inputs(m, 1, n, seed=46)
    nan = np.full((m, n), np.nan + 1j * np.nan)
    C, _ = run_ex("N", "N", 1.5, A, B, 0.0, nan, nmod)                         # beta = 0: NaNs in C are not read
    Cref, D = direct.zgemm_ex_dd("N", "N", 1.5, A, B, 0.0, None)
    assert direct.componentwise_error(C, Cref, D) <= TOL_Z
    C, _ = run_ex("N", "N", 0.0, A * np.nan, B, 2.0 - 1.0j, C0, nmod)          # alpha = 0: C = beta C, A and B not read
    assert np.abs(C - (2.0 - 1.0j) * C0).max() <= 4 * np.spacing(np.abs(C0).max() * 3)
    C, _ = run_ex("N", "N", 0.0, A, B, 0.0, nan, nmod)
    assert (C == 0).all()
    C, _ = run_ex("N", "N", 0.0, A, B, 1.0, C0, nmod)                          # beta = 1: C unchanged
    assert (C == C0).all()


def test_cgemm_extended_and_hybrid_moduli():
    m, n, k = 120, 90, 200
    A, B = inputs.complex_inputs(m, n, k, seed=47, dtype=np.complex64)
    C0, _ = inputs.complex_inputs(m, 1, n, seed=48, dtype=np.complex64)
    alpha, beta = 0.5 + 2.0j, 1.0 - 0.5j
    C, _ = run_ex("T", "C", alpha, A, B, beta, C0, 7, cplx=torch.complex64)
    Cref, D = direct.zgemm_ex_dd("N", "N", alpha, A, B, beta, C0)
    assert C.dtype == np.complex64 and direct.componentwise_error(C, Cref, D) <= TOL_C
    A, B = inputs.complex_inputs(m, n, k, seed=49, dist="phi", phi=3.0)
    C0, _ = inputs.complex_inputs(m, 1, n, seed=50)
    C, _ = run_ex("C", "N", alpha, A, B, beta, C0, 24)                         # 3M planes read in the other orientation too
    Cref, D = direct.zgemm_ex_dd("N", "N", alpha, A, B, beta, C0)
    assert direct.componentwise_error(C, Cref, D) <= TOL_Z


def test_extended_argument_errors():
    A, B = inputs.complex_inputs(8, 8, 8, seed=5)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, 8, 8, 8, 16)):
        C = empty_dev(8, 8, torch.complex128)
        with pytest.raises(b.Gemm2mError, match="ARG"):
            b.zgemm2m_ex("X", "N", None, to_dev(A), to_dev(B), None, C, 16)
        with pytest.raises(ValueError):
            b.zgemm2m_ex("T", "N", None, to_dev(A[:, :5]), to_dev(B), None, C, 16)     # shapes do not fit op(A)

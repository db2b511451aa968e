"""GPU parity of the 2-norm scaling rule (gemm2m_set_scaling(1)) against the staged oracle's integer definition."""
import numpy as np
import pytest
import torch

from oracle import direct, staged
from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host, ulp_distance  # noqa: E402


@pytest.fixture(autouse=True)
def _scaling_mode():
    b.set_scaling(1)
    b.debug_set_gemm_kernel(0)
    yield
    b.set_scaling(0)
    b.debug_set_gemm_kernel(0)


def run(A, B, nmod, cplx=torch.complex128, kernel=0, ta="N", tb="N"):
    m, k = A.shape
    n = B.shape[1]
    op = b.OP_ZGEMM if cplx == torch.complex128 else b.OP_CGEMM
    b.debug_set_gemm_kernel(kernel)
    sto = lambda X, t: np.asfortranarray(X if t == "N" else (X.T if t == "T" else X.conj().T))
    with Workspace(b.workspace_bytes(op, m, n, k, nmod)) as ws:
        C = empty_dev(m, n, cplx)
        fn = b.zgemm2m_ex if op == b.OP_ZGEMM else b.cgemm2m_ex
        fn(ta, tb, None, to_dev(sto(A, ta)), to_dev(sto(B, tb)), None, C, nmod)
        b.device_status()
        return to_host(C), ws.stages(op, m, n, k, nmod)


@pytest.mark.parametrize("shape,nmod,dist,ta,tb", [((200, 150, 300), 16, "phi", "N", "N"), ((129, 257, 1000), 14, "uniform", "T", "N"),
                                                   ((33, 19, 50), 22, "phi", "N", "C"), ((70, 90, 200), 25, "phi", "C", "T"),
                                                   ((64, 64, 2100), 17, "phi", "N", "N"),
                                                   # few moduli: the residue kernel's 32-bit form under this rule (P_A <= 29)
                                                   ((90, 70, 260), 7, "phi", "N", "N"), ((50, 60, 130), 8, "uniform", "C", "N")])
def test_2norm_rule_every_stage(shape, nmod, dist, ta, tb):
    m, n, k = shape
    A, B = inputs.complex_inputs(m, n, k, seed=81, dist=dist, phi=2.0)
    A[1, :] = 0                                       # zero row: exponent 0
    A[2, :] = 0
    A[2, k // 2] = 3.0 - 4.0j                          # a single entry
    A[5, :] *= 2.0 ** -1040                            # subnormal row
    B[:, 3] *= 2.0 ** 600
    C, st = run(A, B, nmod, kernel=1, ta=ta, tb=tb)
    ref = staged.zgemm2m_staged(A, B, nmod, scaling="2norm")
    assert (st["eA"] == ref["eA"]).all() and (st["eB"] == ref["eB"]).all()          # integer rule: bit-exact
    loose = staged.zgemm2m_staged(A, B, nmod, upto="pre")
    assert (ref["eA"] <= loose["eA"]).all() and (ref["eA"] < loose["eA"]).any()
    n2 = min(nmod, 22)
    for j in range(n2):
        for sgn in range(2):
            assert (st["Apm"][sgn, j, :, :k] == ref["Apm"][j][sgn]).all(), ("Apm", sgn, j)
            assert (st["Bpm"][sgn, j, :, :k] == ref["Bpm"][j][sgn].T).all(), ("Bpm", sgn, j)
            assert (st["Cpm"][sgn, j, :, :m] == ref["Cpm"][j][sgn].T).all(), ("Cpm", sgn, j)
    for j3 in range(nmod - n2):
        for part in range(3):
            assert (st["A3"][part, j3, :, :k] == ref["Apm"][22 + j3][part]).all()
            assert (st["C3"][part, j3, :, :m] == ref["Cpm"][22 + j3][part].T).all()
    ok = np.isfinite(ref["C"])
    assert ulp_distance(C.real[ok], ref["C"].real[ok]).max() <= 1 and ulp_distance(C.imag[ok], ref["C"].imag[ok]).max() <= 1


def test_2norm_rule_nonfinite_rows_and_cgemm():
    m, n, k = 90, 70, 400
    A, B = inputs.complex_inputs(m, n, k, seed=82, dtype=np.complex64)
    A[9, 3] = np.inf
    C, st = run(A, B, 8, cplx=torch.complex64)
    assert np.isnan(C[9, :]).all() and np.isfinite(np.delete(C, 9, axis=0)).all()
    ok = np.array([i for i in range(m) if i != 9])
    ref = staged.zgemm2m_staged(A[ok], B, 8, out_bits=24, scaling="2norm")
    assert (st["eA"][ok] == ref["eA"]).all() and (st["eB"] == ref["eB"]).all()
    Cref, D = direct.zgemm4m_dd(A[ok], B)
    assert direct.componentwise_error(C[ok], Cref, D) <= 2e-6


def test_2norm_rule_buys_accuracy_at_the_same_modulus_count():
    m, n, k = 96, 64, 8192                              # long inner dimension: sqrt(2k) = 2^7 is what the max-based rule gives away
    A, B = inputs.complex_inputs(m, n, k, seed=83, dist="phi", phi=0.5)
    Cref, D = direct.zgemm4m_dd(A, B)
    C1, _ = run(A, B, 14)
    b.set_scaling(0)
    C0, _ = run(A, B, 14)
    e0, e1 = direct.componentwise_error(C0, Cref, D), direct.componentwise_error(C1, Cref, D)
    assert e1 * 8 <= e0 and e1 <= 1e-14 < e0

"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: sampled entries against the
double-double oracle and against the exact staged integers, plus full-coverage properties."""
import numpy as np
import pytest
import torch

from oracle import direct, staged
from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host, ulp_distance  # noqa: E402


def staged_for_pairs(A, B, nmod, pairs, herk=False, out_bits=53):
    """Staged oracle restricted to the rows of A / columns of B that the sampled entries touch (scale factors are
    per row / per column, so the restriction changes nothing)."""
    rows, ri = np.unique(pairs[:, 0], return_inverse=True)
    cols, ci = np.unique(pairs[:, 1], return_inverse=True)
    st = staged.zgemm2m_staged(A[rows, :], B[:, cols], nmod, herk=herk, upto="pre")
    sub = np.stack([ri, ci], axis=1)
    Xs, vals = staged.staged_samples(st, sub, out_bits=out_bits)
    return st, rows, cols, vals


@pytest.mark.parametrize("phi,nmod,tol", [(0.5, 16, 1e-14), (1.0, 16, 1e-14), (2.0, 18, 1e-14)])
def test_zgemm_8192_sampled(phi, nmod, tol):
    m = n = k = 8192
    A, B = inputs.complex_inputs(m, n, k, seed=1, dist="phi", phi=phi)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, nmod)) as ws:
        C = empty_dev(m, n, torch.complex128)
        b.zgemm2m(to_dev(A), to_dev(B), C, nmod)
        b.device_status()
        lay = b.workspace_layout(b.OP_ZGEMM, m, n, k, nmod)
        eA = ws.buf[lay["off_exp_a"]: lay["off_exp_a"] + 4 * m].cpu().numpy().view(np.int32)
        eB = ws.buf[lay["off_exp_b"]: lay["off_exp_b"] + 4 * n].cpu().numpy().view(np.int32)
        C = to_host(C)
    assert np.isfinite(C.real).all() and np.isfinite(C.imag).all()
    pairs = inputs.sample_indices(m, n, 4096, seed=3, tile=128)
    Cs, Ds = direct.zgemm4m_dd_samples(A, B, pairs)
    got = C[pairs[:, 0], pairs[:, 1]]
    assert direct.componentwise_error(got, Cs, Ds) <= tol
    # exact staged integers on a smaller sample: the GPU value is the correctly rounded lifted integer (<= 1 ulp)
    sub = pairs[:256]
    st, rows, cols, vals = staged_for_pairs(A, B, nmod, sub)
    assert (eA[rows] == st["eA"]).all() and (eB[cols] == st["eB"]).all()
    g = C[sub[:, 0], sub[:, 1]]
    assert ulp_distance(g.real, vals.real).max() <= 1 and ulp_distance(g.imag, vals.imag).max() <= 1
    # full coverage: the scale exponents follow the closed-form rule for every row and column
    M = staged.product(staged.greedy_2m_moduli()[:nmod])
    Pt, PA, PB, ck = staged.scaling_targets(M, k)
    assert (eA == staged.scaling_exponents(A, 1, PA, ck)).all() and (eB == staged.scaling_exponents(B, 0, PB, ck)).all()


def test_cgemm_16384_sampled():
    m = n = 16384
    k = 4096
    A, B = inputs.complex_inputs(m, n, k, seed=1, dtype=np.complex64)
    with Workspace(b.workspace_bytes(b.OP_CGEMM, m, n, k, 7)):
        C = empty_dev(m, n, torch.complex64)
        b.cgemm2m(to_dev(A), to_dev(B), C, 7)
        b.device_status()
        pairs = inputs.sample_indices(m, n, 4096, seed=4, tile=128)
        idx = torch.from_numpy(pairs).cuda()
        got = C[idx[:, 0], idx[:, 1]].cpu().numpy()
        finite = bool(torch.isfinite(torch.view_as_real(C)).all())
    assert finite
    Cs, Ds = direct.zgemm4m_dd_samples(A, B, pairs)
    assert direct.componentwise_error(got, Cs, Ds) <= 2e-6


def test_zherk_8192_sampled():
    n = k = 8192
    A = inputs.herk_input(n, k, seed=1)
    with Workspace(b.workspace_bytes(b.OP_ZHERK, n, n, k, 16)):
        C = empty_dev(n, n, torch.complex128, fill=-5.0)
        b.zherk2m(to_dev(A), C, 16)
        b.device_status()
        pairs = inputs.sample_indices(n, n, 4096, seed=5, tile=128)
        pairs = np.stack([np.maximum(pairs[:, 0], pairs[:, 1]), np.minimum(pairs[:, 0], pairs[:, 1])], axis=1)   # lower triangle
        idx = torch.from_numpy(pairs).cuda()
        got = C[idx[:, 0], idx[:, 1]].cpu().numpy()
        upper_ok = bool((torch.triu(C.real, diagonal=1) == torch.triu(torch.full_like(C.real, -5.0), diagonal=1)).all())
        diag_imag_zero = bool((torch.diagonal(C).imag == 0).all())
    assert upper_ok and diag_imag_zero
    AH = np.asfortranarray(A.conj().T)
    Cs, Ds = direct.zgemm4m_dd_samples(A, AH, pairs)
    assert direct.componentwise_error(got, Cs, Ds) <= 1e-14

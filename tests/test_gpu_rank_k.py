"""GPU parity of the rank-k family of Section 5 (HER2K, SYRK, SYR2K) against the oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from oracle import direct, staged
from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host, ulp_distance  # noqa: E402

TOL = 1e-14


def real_input(n, k, seed, dist="uniform", phi=0.5):
    return np.asfortranarray(inputs.herk_input(n, k, seed, dist, phi).real.copy())


def stages_rank(ws, op, n, k, nmod):
    torch.cuda.synchronize()
    lay = b.workspace_layout(op, n, n, k, nmod)
    raw = ws.buf.cpu().numpy()
    eA = raw[lay["off_exp_a"]: lay["off_exp_a"] + 4 * n].view(np.int32).copy()
    cp = raw[lay["off_cpm"]: lay["off_cpm"] + nmod * n * lay["ldp"]].view(np.int8).reshape(nmod, n, lay["ldp"])
    return eA, cp


@pytest.mark.parametrize("kernel", [1, 0], ids=["checkgemm", "tcgen05"])
@pytest.mark.parametrize("n,k,nmod", [(96, 200, 16), (257, 129, 16), (130, 70, 18), (64, 40, 21)])
def test_zher2k_parity(n, k, nmod, kernel):
    A = inputs.herk_input(n, k, seed=31, dist="phi", phi=1.0)
    B = inputs.herk_input(n, k, seed=32, dist="phi", phi=1.0)
    b.debug_set_gemm_kernel(kernel)
    try:
        with Workspace(b.workspace_bytes(b.OP_ZHER2K, n, n, k, nmod)) as ws:
            C = empty_dev(n, n, torch.complex128, fill=-5.0)
            b.zher2k2m(to_dev(A), to_dev(B), C, nmod)
            b.device_status()
            eA, cp = stages_rank(ws, b.OP_ZHER2K, n, k, nmod)
            Ch = to_host(C)
    finally:
        b.debug_set_gemm_kernel(0)
    ref = staged.zher2k2m_staged(A, B, nmod)
    assert (eA == ref["eA"]).all()                                              # sigma = tau: one scale vector
    for j in range(nmod):
        assert (cp[j, :, :n] == ref["Cpm"][j][0].T).all(), j                    # C+ = A+ B-^T + B+ A-^T (mod m_j)
    low = np.tril(np.ones((n, n), dtype=bool))
    assert (Ch[~low] == -5.0).all() and (np.diag(Ch).imag == 0).all()
    assert ulp_distance(Ch[low].real, ref["C"][low].real).max() <= 1 and ulp_distance(Ch[low].imag, ref["C"][low].imag).max() <= 1
    Cref, D = direct.zher2k_dd(A, B)
    if nmod >= 17:
        assert direct.componentwise_error(Ch[low], Cref[low], D[low]) <= TOL
    else:
        assert direct.componentwise_error(Ch[low], Cref[low], D[low]) <= 4 * TOL    # one bit less per operand than HERK at the same N


@pytest.mark.parametrize("n,k,nmod", [(96, 200, 16), (130, 301, 16), (257, 1, 16), (64, 75, 20)])
def test_dsyrk_parity(n, k, nmod):
    A = real_input(n, k, seed=33, dist="phi", phi=1.0)
    with Workspace(b.workspace_bytes(b.OP_DSYRK, n, n, k, nmod)) as ws:
        C = empty_dev(n, n, torch.float64, fill=-5.0)
        b.dsyrk2m(to_dev(A), C, nmod)
        b.device_status()
        eA, cp = stages_rank(ws, b.OP_DSYRK, n, k, nmod)
        Ch = to_host(C)
    Z = staged.syrk_complexify(A)                                               # Section 5: SYRK = Re(HERK(A1 + i A2))
    ref = staged.zgemm2m_staged(Z, np.asfortranarray(Z.conj().T), nmod, herk=True)
    assert (eA == ref["eA"]).all()
    for j in range(nmod):
        assert (cp[j, :, :n] == ref["Cpm"][j][0].T).all(), j
    low = np.tril(np.ones((n, n), dtype=bool))
    assert (Ch[~low] == -5.0).all()
    assert ulp_distance(Ch[low], ref["C"].real[low]).max() <= 1
    Cref, D = direct.dsyrk_dd(A)
    assert direct.componentwise_error(Ch[low], Cref[low], D[low]) <= TOL


@pytest.mark.parametrize("n,k,nmod", [(96, 200, 17), (130, 33, 17)])
def test_dsyr2k_parity(n, k, nmod):
    A = real_input(n, k, seed=34)
    B = real_input(n, k, seed=35)
    with Workspace(b.workspace_bytes(b.OP_DSYR2K, n, n, k, nmod)) as ws:
        C = empty_dev(n, n, torch.float64, fill=-5.0)
        b.dsyr2k2m(to_dev(A), to_dev(B), C, nmod)
        b.device_status()
        eA, cp = stages_rank(ws, b.OP_DSYR2K, n, k, nmod)
        Ch = to_host(C)
    ref = staged.zher2k2m_staged(staged.syrk_complexify(A), staged.syrk_complexify(B), nmod)
    assert (eA == ref["eA"]).all()
    for j in range(nmod):
        assert (cp[j, :, :n] == ref["Cpm"][j][0].T).all(), j
    low = np.tril(np.ones((n, n), dtype=bool))
    assert (Ch[~low] == -5.0).all()
    assert ulp_distance(Ch[low], ref["C"].real[low]).max() <= 1
    Cref, D = direct.dsyr2k_dd(A, B)
    assert direct.componentwise_error(Ch[low], Cref[low], D[low]) <= TOL


def test_rank_k_at_size_sampled():
    n, k = 4096, 4096
    A = real_input(n, k, seed=36)
    with Workspace(b.workspace_bytes(b.OP_DSYRK, n, n, k, 16)):
        C = empty_dev(n, n, torch.float64, fill=-5.0)
        b.dsyrk2m(to_dev(A), C, 16)
        b.device_status()
        Ch = to_host(C)
    pairs = inputs.sample_indices(n, n, 2048, seed=6, tile=128)
    pairs = np.stack([np.maximum(pairs[:, 0], pairs[:, 1]), np.minimum(pairs[:, 0], pairs[:, 1])], axis=1)
    Az = A.astype(np.complex128)
    Cs, Ds = direct.zgemm4m_dd_samples(Az, np.asfortranarray(Az.T), pairs)
    assert direct.componentwise_error(Ch[pairs[:, 0], pairs[:, 1]], Cs.real, Ds) <= TOL
    assert (np.triu(Ch, 1)[np.triu(np.ones((n, n), dtype=bool), 1)] == -5.0).all()


def test_rank_k_row_panels_are_bitwise_identical():
    """The rank-k family cuts the output into row panels and post-processes panel p beside the GEMMs of panel p + 1: the
    result must not depend on the number of panels, the upper triangle stays untouched, and work queued on the caller's
    stream right after the call sees the whole result."""
    n, k, nmod = 2304, 96, 16                      # 2304 rows -> 2 panels of 1280 / 1024
    A = inputs.herk_input(n, k, seed=51, dist="phi", phi=1.0)
    B = inputs.herk_input(n, k, seed=52, dist="phi", phi=1.0)
    X = real_input(n, k, seed=53)
    dA, dB, dX = to_dev(A), to_dev(B), to_dev(X)
    results = {}
    try:
        with Workspace(max(b.workspace_bytes(b.OP_ZHER2K, n, n, k, nmod), b.workspace_bytes(b.OP_DSYRK, n, n, k, nmod))):
            for panels in (1, 8):
                b.debug_set_panels(panels)
                C1 = empty_dev(n, n, torch.complex128, fill=-5.0)
                C2 = empty_dev(n, n, torch.complex128, fill=-5.0)
                C3 = empty_dev(n, n, torch.float64, fill=-5.0)
                b.zherk2m(dA, C1, nmod)
                snap = C1.clone()                  # same stream, no synchronisation in between
                if panels == 8:
                    assert b.last_launch_count()[1][2:] == [2, 2]      # one GEMM and one post launch per panel
                b.zher2k2m(dA, dB, C2, nmod)
                b.dsyrk2m(dX, C3, nmod)
                b.device_status()
                assert (to_host(snap) == to_host(C1)).all()
                results[panels] = (to_host(C1), to_host(C2), to_host(C3))
    finally:
        b.debug_set_panels(8)
    for a, c in zip(results[1], results[8]):
        assert (a == c).all()
    C1, C2, C3 = results[8]
    iu = np.triu_indices(n, 1)
    assert (C1[iu] == -5.0).all() and (C2[iu] == -5.0).all() and (C3[iu] == -5.0).all()
    il = np.tril_indices(n)
    pairs = np.stack([il[0], il[1]], axis=1)[:: 997]                            # a sample of the lower triangle, all panels
    Cs, Ds = direct.zgemm4m_dd_samples(A, A.conj().T, pairs)
    assert direct.componentwise_error(C1[pairs[:, 0], pairs[:, 1]], Cs, Ds) <= TOL
    Cs, Ds = direct.zgemm4m_dd_samples(X.astype(np.complex128), X.T.astype(np.complex128), pairs)
    assert direct.componentwise_error(C3[pairs[:, 0], pairs[:, 1]] + 0j, Cs, Ds) <= TOL

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


def test_extensions_4096_sampled():
    """The later entry points at a size that spans many tiles, panels and waves: hybrid moduli, transposed / conjugated
    operands with alpha and beta, the 2-norm scaling rule and the real scheme, each on sampled entries against the
    double-double definition (and, for the hybrid, against the exact staged integers)."""
    m = n = k = 4096
    A, B = inputs.complex_inputs(m, n, k, seed=5, dist="phi", phi=2.0)
    pairs = inputs.sample_indices(m, n, 2048, seed=6, tile=128)
    idx = torch.from_numpy(pairs).cuda()
    Cs, Ds = direct.zgemm4m_dd_samples(A, B, pairs)
    dA, dB = to_dev(A), to_dev(B)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, 24)):
        C = empty_dev(m, n, torch.complex128)
        # hybrid 2M/3M, 24 moduli: 50 planes per operand
        b.zgemm2m(dA, dB, C, 24)
        b.device_status()
        got = C[idx[:, 0], idx[:, 1]].cpu().numpy()
        assert direct.componentwise_error(got, Cs, Ds) <= 1e-14
        sub = pairs[:128]
        rows, ri = np.unique(sub[:, 0], return_inverse=True)
        cols, ci = np.unique(sub[:, 1], return_inverse=True)
        st = staged.zgemm2m_staged(A[rows, :], B[:, cols], 24, upto="pre")
        _, vals = staged.staged_samples(st, np.stack([ri, ci], axis=1))
        g = got[:128]
        assert ulp_distance(g.real, vals.real).max() <= 1 and ulp_distance(g.imag, vals.imag).max() <= 1
        # C = alpha A^H^H B^T^T + beta C with the operands stored conjugate-transposed / transposed
        alpha, beta = 0.5 - 2.0j, 1.5 + 0.25j
        C0 = C.clone()
        c0 = C0[idx[:, 0], idx[:, 1]].cpu().numpy()
        dAh = to_dev(np.asfortranarray(A.conj().T))
        dBt = to_dev(np.asfortranarray(B.T))
        b.zgemm2m_ex("C", "T", alpha, dAh, dBt, beta, C, 18)
        b.device_status()
        got = C[idx[:, 0], idx[:, 1]].cpu().numpy()
        want = alpha * Cs.astype(np.clongdouble) + beta * c0.astype(np.clongdouble)
        scale = abs(alpha) * Ds + abs(beta) * np.abs(c0)
        assert (np.abs(got - want.astype(np.complex128)) <= 1e-14 * scale).all()
        # 2-norm scaling rule: 16 moduli reach 1e-14 for this exponent spread, where the max-based rule needs 18
        b.set_scaling(1)
        try:
            b.zgemm2m(dA, dB, C, 16)
            b.device_status()
        finally:
            b.set_scaling(0)
        e2 = direct.componentwise_error(C[idx[:, 0], idx[:, 1]].cpu().numpy(), Cs, Ds)
        b.zgemm2m(dA, dB, C, 16)
        b.device_status()
        e0 = direct.componentwise_error(C[idx[:, 0], idx[:, 1]].cpu().numpy(), Cs, Ds)
        assert e2 < e0 and e2 <= 1e-14
    # real Ozaki-II scheme
    Ar, Br = np.asfortranarray(A.real.copy()), np.asfortranarray(B.real.copy())
    with Workspace(b.workspace_bytes(b.OP_DGEMM_OZAKI2, m, n, k, 17)):
        Cr = empty_dev(m, n, torch.float64)
        b.dgemm_ozaki2(to_dev(Ar), to_dev(Br), Cr, 17)
        b.device_status()
        got = Cr[idx[:, 0], idx[:, 1]].cpu().numpy()
    Cd, Dd = direct.zgemm4m_dd_samples(Ar.astype(np.complex128), Br.astype(np.complex128), pairs)
    assert direct.componentwise_error(got + 0j, Cd, Dd) <= 1e-14


def test_zgemm_8192_full_coverage_of_every_stage():
    """Every element of every plane at the benchmark's size: (a) the residue planes of A for two moduli against the oracle's
    quantiser and Eq. (2a) on all 67 M entries, and for all moduli on sampled rows of A and columns of B; (b) Eq. (2b) on all
    2N planes by a Freivalds check modulo m_j: Cpm X = Bpm (Apm^T X) (mod m_j) for four random vectors X, computed exactly in
    float64 (all partial sums stay below 2^31).  A wrong entry of a product plane escapes a vector with probability at most
    1/p, p the smallest prime factor of m_j; (c) the final C on all entries through C x = A (B x) in extended precision."""
    m = n = k = 8192
    nmod = 16
    A, B = inputs.complex_inputs(m, n, k, seed=1, dist="phi", phi=0.5)
    moduli = staged.greedy_2m_moduli()[:nmod]
    roots = staged.roots_of(moduli)
    M = staged.product(moduli)
    Pt, PA, PB, ck = staged.scaling_targets(M, k)
    eA, eB = staged.scaling_exponents(A, 1, PA, ck), staged.scaling_exponents(B, 0, PB, ck)
    rng = np.random.default_rng(5)
    X = rng.integers(0, 1024, (m, 4)).astype(np.float64)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, nmod)) as ws:
        C = empty_dev(m, n, torch.complex128)
        b.zgemm2m(to_dev(A), to_dev(B), C, nmod)
        b.device_status()
        lay = b.workspace_layout(b.OP_ZGEMM, m, n, k, nmod)
        kp, ldp = lay["kp"], lay["ldp"]
        assert kp == k and ldp == m
        Cfull = to_host(C)

        def plane(off, rows, ld, idx):
            lo = off + idx * rows * ld
            return ws.buf[lo: lo + rows * ld].cpu().numpy().view(np.int8).reshape(rows, ld)

        assert (ws.buf[lay["off_exp_a"]: lay["off_exp_a"] + 4 * m].cpu().numpy().view(np.int32) == eA).all()
        assert (ws.buf[lay["off_exp_b"]: lay["off_exp_b"] + 4 * n].cpu().numpy().view(np.int32) == eB).all()
        # (b) Eq. (2b), every plane
        for sgn in range(2):
            for j, mj in enumerate(moduli):
                idx = sgn * nmod + j
                Ap = plane(lay["off_apm"], m, kp, idx).astype(np.float64)
                Bp = plane(lay["off_bpm"], n, kp, idx).astype(np.float64)
                Cp = plane(lay["off_cpm"], n, ldp, idx).astype(np.float64)     # Cp[col, row] = C+-[row, col]
                assert np.abs(Ap).max() <= (mj - 1) // 2 and np.abs(Bp).max() <= (mj - 1) // 2 and np.abs(Cp).max() <= (mj - 1) // 2
                inner = np.mod(Ap.T @ X, mj)                                    # (k x 4), entries < 2^31 before the reduction
                assert np.array_equal(np.mod(Cp @ X, mj), np.mod(Bp @ inner, mj)), (sgn, j)
        # (a) steps 3-4 on every entry of A for the first and the last modulus ...
        Ar, Ai = staged.quantise(A, eA, 1, int64_ok=True)
        assert Ar.dtype == np.int64
        for j in (0, nmod - 1):
            want = staged.pre_2m(Ar % moduli[j], Ai % moduli[j], moduli[j], roots[j])
            for sgn in range(2):
                assert np.array_equal(plane(lay["off_apm"], m, kp, sgn * nmod + j), want[sgn]), (sgn, j)
        # ... and for every modulus on sampled rows of A and columns of B
        rows = np.unique(np.concatenate([rng.integers(0, m, 96), [0, 1, 127, 128, m - 1]]))
        Br, Bi = staged.quantise(B[:, rows], eB[rows], 0, int64_ok=True)
        for j, mj in enumerate(moduli):
            wa = staged.pre_2m(Ar[rows] % mj, Ai[rows] % mj, mj, roots[j])
            wb = staged.pre_2m(Br % mj, Bi % mj, mj, roots[j])
            for sgn in range(2):
                assert np.array_equal(plane(lay["off_apm"], m, kp, sgn * nmod + j)[rows], wa[sgn]), ("A", sgn, j)
                assert np.array_equal(plane(lay["off_bpm"], n, kp, sgn * nmod + j)[rows], wb[sgn].T), ("B", sgn, j)
    # (c) steps 5-7, every entry of C, as a net for gross errors: C x = A (B x) for a random +-1 vector x, the right-hand side in
    # extended precision.  An entry of C that is off by more than about 1e-10 |A||B| would show in its row.
    L = np.clongdouble
    x = rng.choice([-1.0, 1.0], n)
    y = np.zeros(k, dtype=L)
    for c0 in range(0, n, 1024):
        y += B[:, c0:c0 + 1024].astype(L) @ x[c0:c0 + 1024].astype(L)
    lhs, rhs, scale = np.zeros(m, dtype=L), np.zeros(m, dtype=L), np.zeros(m)
    absBx = np.abs(B) @ np.ones(n)
    for c0 in range(0, k, 1024):
        rhs += A[:, c0:c0 + 1024].astype(L) @ y[c0:c0 + 1024]
        scale += np.abs(A[:, c0:c0 + 1024]) @ absBx[c0:c0 + 1024]
    for c0 in range(0, n, 1024):
        lhs += Cfull[:, c0:c0 + 1024].astype(L) @ x[c0:c0 + 1024].astype(L)
    assert np.max(np.abs(lhs - rhs).astype(np.float64) / scale) < 1e-14

"""GPU parity tests: the CUDA path, called through the C-ABI, against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import direct, staged
from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host, ulp_distance  # noqa: E402

TOL_Z = 1e-14      # complex128: max |C - Cref| / (|A||B|)
TOL_C = 2e-6       # complex64


@pytest.fixture(autouse=True)
def _default_kernel():
    b.debug_set_gemm_kernel(0)
    b.debug_set_panels(8)
    b.debug_set_overlap(False)
    b.debug_set_chained_launch(True)
    yield
    b.debug_set_gemm_kernel(0)
    b.debug_set_panels(8)
    b.debug_set_overlap(False)
    b.debug_set_chained_launch(True)


def run_int(Ar, Ai, Br, Bi, nmod, kernel=0, ldc=None):
    m, k = Ar.shape
    n = Br.shape[1]
    b.debug_set_gemm_kernel(kernel)
    with Workspace(b.workspace_bytes(b.OP_GAUSSIAN_INT, m, n, k, nmod)) as ws:
        Cr = empty_dev(m, n, torch.int64, ld=ldc, fill=-7)
        Ci = empty_dev(m, n, torch.int64, ld=ldc, fill=-7)
        b.gemm2m_gaussian_int(to_dev(Ar), to_dev(Ai), to_dev(Br), to_dev(Bi), Cr, Ci, nmod)
        b.device_status()
        st = ws.stages(b.OP_GAUSSIAN_INT, m, n, k, nmod)
        return to_host(Cr), to_host(Ci), st


def check_stages_int(st, ref, m, n, k, nmod):
    for j in range(nmod):
        for sgn in range(2):
            assert (st["Apm"][sgn, j, :, :k] == ref["Apm"][j][sgn]).all(), ("Apm", sgn, j)
            assert (st["Bpm"][sgn, j, :, :k] == ref["Bpm"][j][sgn].T).all(), ("Bpm", sgn, j)
            assert (st["Apm"][sgn, j, :, k:] == 0).all() and (st["Bpm"][sgn, j, :, k:] == 0).all()
            assert (st["Cpm"][sgn, j, :, :m] == ref["Cpm"][j][sgn].T).all(), ("Cpm", sgn, j)


@pytest.mark.parametrize("kernel", [1, 0], ids=["checkgemm", "tcgen05"])   # check kernel first: isolates pre/post from the tensor-core GEMM
@pytest.mark.parametrize("shape,nmod", [((128, 128, 128), 3), ((128, 128, 128), 1), ((128, 128, 128), 2),
                                        ((130, 77, 300), 3), ((1, 1, 1), 1), ((257, 513, 129), 4), ((5, 300, 1000), 8)])
def test_gaussian_int_bit_exact(shape, nmod, kernel):
    m, n, k = shape
    full = nmod == 8
    Ar, Ai, Br, Bi = inputs.gaussian_int_inputs(m, n, k, seed=1 + nmod, lo=-128 if full else -16, hi=127 if full else 16)
    Cr, Ci, st = run_int(Ar, Ai, Br, Bi, nmod, kernel)
    M = staged.product(staged.greedy_2m_moduli()[:nmod])
    er, ei = direct.gauss4m_mod(Ar, Ai, Br, Bi, M)
    ref = staged.gemm2m_int_staged(Ar, Ai, Br, Bi, nmod)
    check_stages_int(st, ref, m, n, k, nmod)
    assert (Cr == er).all() and (Ci == ei).all()


def test_gaussian_int_padded_leading_dimensions_and_untouched_padding():
    m, n, k = 70, 45, 200
    Ar, Ai, Br, Bi = inputs.gaussian_int_inputs(m, n, k, seed=21)
    pad = lambda a, ld: np.asfortranarray(np.vstack([a, np.full((ld - a.shape[0], a.shape[1]), 99, dtype=a.dtype)]))
    with Workspace(b.workspace_bytes(b.OP_GAUSSIAN_INT, m, n, k, 3)):
        dAr, dAi = to_dev(pad(Ar, 80))[:m], to_dev(pad(Ai, 80))[:m]
        dBr, dBi = to_dev(pad(Br, 256))[:k], to_dev(pad(Bi, 256))[:k]
        Crf = empty_dev(96, n, torch.int64, fill=-7)
        Cif = empty_dev(96, n, torch.int64, fill=-7)
        b.gemm2m_gaussian_int(dAr, dAi, dBr, dBi, Crf[:m], Cif[:m], 3)
        b.device_status()
        Cr, Ci = to_host(Crf), to_host(Cif)
    er, ei = direct.gauss4m_mod(Ar, Ai, Br, Bi, staged.product(staged.greedy_2m_moduli()[:3]))
    assert (Cr[:m] == er).all() and (Ci[:m] == ei).all()
    assert (Cr[m:] == -7).all() and (Ci[m:] == -7).all()


def test_gaussian_int_k_split_beyond_int32_range():
    # k ((241-1)/2)^2 > 2^31: the GEMM must split K and add residues; extreme entries make the overflow real
    m, n, k = 40, 24, 150000 + 77
    Ar = np.asfortranarray(np.full((m, k), 120, dtype=np.int8))
    Ai = np.asfortranarray(np.zeros((m, k), dtype=np.int8))
    Br = np.asfortranarray(np.full((k, n), 120, dtype=np.int8))
    Bi = np.asfortranarray(np.zeros((k, n), dtype=np.int8))
    rng = np.random.default_rng(5)
    Ar[:, ::7] = rng.integers(-128, 128, size=Ar[:, ::7].shape)
    Bi[::5, :] = rng.integers(-128, 128, size=Bi[::5, :].shape)
    M = staged.product(staged.greedy_2m_moduli()[:6])
    er, ei = direct.gauss4m_mod(Ar, Ai, Br, Bi, M)
    for kernel in (1, 0):
        Cr, Ci, _ = run_int(Ar, Ai, Br, Bi, 6, kernel)
        assert (Cr == er).all() and (Ci == ei).all(), kernel


def run_z(A, B, nmod, kernel=0, cplx=torch.complex128, op=None):
    m, k = A.shape
    n = B.shape[1]
    op = op or (b.OP_ZGEMM if cplx == torch.complex128 else b.OP_CGEMM)
    b.debug_set_gemm_kernel(kernel)
    with Workspace(b.workspace_bytes(op, m, n, k, nmod)) as ws:
        C = empty_dev(m, n, cplx)
        (b.zgemm2m if op == b.OP_ZGEMM else b.cgemm2m)(to_dev(A), to_dev(B), C, nmod)
        b.device_status()
        st = ws.stages(op, m, n, k, nmod) if m * n * k else None
        return to_host(C), st


@pytest.mark.parametrize("kernel", [1, 0], ids=["checkgemm", "tcgen05"])
@pytest.mark.parametrize("shape,nmod,dist", [((200, 150, 300), 16, "phi"), ((129, 257, 128), 14, "uniform"),
                                             ((64, 64, 64), 3, "uniform"), ((33, 19, 50), 22, "phi"), ((40, 40, 520), 20, "uniform"),
                                             # few moduli: quantised parts below 2^31 take the residue kernel's 32-bit path
                                             ((96, 80, 260), 8, "phi"), ((50, 70, 90), 7, "uniform"), ((70, 33, 130), 10, "phi"),
                                             ((33, 70, 40), 11, "uniform")])
def test_zgemm_every_stage_against_staged_oracle(shape, nmod, dist, kernel):
    m, n, k = shape
    A, B = inputs.complex_inputs(m, n, k, seed=7, dist=dist, phi=1.0)
    C, st = run_z(A, B, nmod, kernel)
    ref = staged.zgemm2m_staged(A, B, nmod)
    assert (st["eA"] == ref["eA"]).all() and (st["eB"] == ref["eB"]).all()          # step 2: integer rule, bit-exact
    for j in range(nmod):
        for sgn in range(2):
            assert (st["Apm"][sgn, j, :, :k] == ref["Apm"][j][sgn]).all(), ("Apm", sgn, j)       # steps 3-4, Eq. (2a)
            assert (st["Bpm"][sgn, j, :, :k] == ref["Bpm"][j][sgn].T).all(), ("Bpm", sgn, j)
            assert (st["Cpm"][sgn, j, :, :m] == ref["Cpm"][j][sgn].T).all(), ("Cpm", sgn, j)     # Eq. (2b)
    # steps 5-7: at most one unit in the last place from the exactly rounded value (identical except near ties)
    assert ulp_distance(C.real, ref["C"].real).max() <= 1 and ulp_distance(C.imag, ref["C"].imag).max() <= 1
    assert (C == ref["C"]).mean() > 0.999
    Cref, D = direct.zgemm4m_dd(A, B)
    if nmod >= 16:
        assert direct.componentwise_error(C, Cref, D) <= TOL_Z


@pytest.mark.parametrize("kernel", [1, 0], ids=["checkgemm", "tcgen05"])
@pytest.mark.parametrize("shape,nmod,phi", [((70, 90, 200), 23, 4.0), ((129, 257, 128), 26, 6.0), ((33, 19, 50), 24, 1.0),
                                            ((40, 300, 520), 25, 8.0)])
def test_zgemm_hybrid_every_stage_against_staged_oracle(shape, nmod, phi, kernel):
    """Hybrid 2M/3M (Section 3 remark): the moduli beyond the 22nd take Eq. (1) with three planes each."""
    m, n, k = shape
    A, B = inputs.complex_inputs(m, n, k, seed=17, dist="phi", phi=phi)       # wide exponent span: what the hybrid is for
    C, st = run_z(A, B, nmod, kernel)
    ref = staged.zgemm2m_staged(A, B, nmod)
    assert (st["eA"] == ref["eA"]).all() and (st["eB"] == ref["eB"]).all()
    for j in range(22):
        for sgn in range(2):
            assert (st["Apm"][sgn, j, :, :k] == ref["Apm"][j][sgn]).all(), ("Apm", sgn, j)
            assert (st["Bpm"][sgn, j, :, :k] == ref["Bpm"][j][sgn].T).all(), ("Bpm", sgn, j)
            assert (st["Cpm"][sgn, j, :, :m] == ref["Cpm"][j][sgn].T).all(), ("Cpm", sgn, j)
    for j3 in range(nmod - 22):
        for part in range(3):                                                  # X_r, X_i, X_r + X_i  /  P1, P2, P3
            assert (st["A3"][part, j3, :, :k] == ref["Apm"][22 + j3][part]).all(), ("A3", part, j3)
            assert (st["B3"][part, j3, :, :k] == ref["Bpm"][22 + j3][part].T).all(), ("B3", part, j3)
            assert (st["C3"][part, j3, :, :m] == ref["Cpm"][22 + j3][part].T).all(), ("C3", part, j3)
    assert ulp_distance(C.real, ref["C"].real).max() <= 1 and ulp_distance(C.imag, ref["C"].imag).max() <= 1
    assert (C == ref["C"]).mean() > 0.999
    Cref, D = direct.zgemm4m_dd(A, B)
    err = direct.componentwise_error(C, Cref, D)
    if phi <= 4.0:
        assert err <= TOL_Z
    else:       # the spread of exponents inside a row exceeds what any M <= 2^184 resolves: the method's own limit, which
        assert err <= 1.01 * direct.componentwise_error(ref["C"], Cref, D)      # the staged oracle shares


def test_hybrid_k_split_with_the_even_modulus():
    """k 128^2 > 2^31 once the modulus 256 is in use: the split point moves to 130 944 and the second K chunk is added to
    the stored residues in the epilogue, for the 3M planes and the even modulus too.  Rows whose quantised entries are
    all +-2^j make every residue of 256 equal to 0 or -128 (the corner of its range) where the digit weight allows."""
    m, n, k, nmod = 24, 40, 131072 + 300, 23
    A, B = inputs.complex_inputs(m, n, k, seed=61, dist="phi", phi=1.5)
    A[3, :] = (2.0 ** 40) * (1 + 1j)                   # constant rows / columns: quantise to the same integer everywhere
    B[:, 5] = -(2.0 ** -17) * (1 - 1j)
    ref = staged.zgemm2m_staged(A, B, nmod)
    for kernel in (1, 0):
        C, st = run_z(A, B, nmod, kernel)
        for j3 in range(nmod - 22):
            for part in range(3):
                assert (st["C3"][part, j3, :, :m] == ref["Cpm"][22 + j3][part].T).all(), ("C3", part, j3, kernel)
        for j in (0, 21):
            for sgn in range(2):
                assert (st["Cpm"][sgn, j, :, :m] == ref["Cpm"][j][sgn].T).all(), ("Cpm", sgn, j, kernel)
        assert ulp_distance(C.real, ref["C"].real).max() <= 1 and ulp_distance(C.imag, ref["C"].imag).max() <= 1


def test_hybrid_beats_the_2m_set_on_a_wide_exponent_span_and_cgemm_accepts_it():
    m, n, k = 48, 40, 160
    A, B = inputs.complex_inputs(m, n, k, seed=23, dist="phi", phi=6.0)    # all 22 2M moduli fall short of double precision here
    Cref, D = direct.zgemm4m_dd(A, B)
    e22 = direct.componentwise_error(run_z(A, B, 22)[0], Cref, D)
    e26 = direct.componentwise_error(run_z(A, B, 26)[0], Cref, D)
    assert e22 > 1e-13 and e26 <= TOL_Z
    A32, B32 = A.astype(np.complex64), B.astype(np.complex64)
    C32, _ = run_z(A32, B32, 23, cplx=torch.complex64)
    ref = staged.zgemm2m_staged(A32, B32, 23, out_bits=24)
    for got, want in ((C32.real, ref["C"].real), (C32.imag, ref["C"].imag)):   # 53 then 24 bits: within one float ulp
        assert (np.abs(got.astype(np.float64) - want) <= np.spacing(np.abs(want).astype(np.float32)).astype(np.float64)).all()


@pytest.mark.parametrize("nmod,tol", [(16, TOL_Z), (15, TOL_Z), (14, 1e-13)])
def test_zgemm_1024_full_oracle(nmod, tol):
    A, B = inputs.complex_inputs(1024, 1024, 1024, seed=1)
    C, _ = run_z(A, B, nmod)
    Cref, D = direct.zgemm4m_dd(A, B)
    assert direct.componentwise_error(C, Cref, D) <= tol


def test_zgemm_ragged_and_padded():
    m, n, k = 333, 130, 257
    A, B = inputs.complex_inputs(m, n, k, seed=3, dist="phi", phi=2.0)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, 18)):
        Af = to_dev(np.asfortranarray(np.vstack([A, np.full((7, k), np.nan)])))
        Bf = to_dev(np.asfortranarray(np.vstack([B, np.full((3, n), np.inf)])))
        Cf = empty_dev(m + 5, n, torch.complex128, fill=-3.0)
        b.zgemm2m(Af[:m], Bf[:k], Cf[:m], 18)
        b.device_status()
        C = to_host(Cf)
    Cref, D = direct.zgemm4m_dd(A, B)
    assert direct.componentwise_error(C[:m], Cref, D) <= TOL_Z
    assert (C[m:] == -3.0).all()


def test_zgemm_degenerate_inputs():
    m, n, k = 70, 50, 90
    A, B = inputs.complex_inputs(m, n, k, seed=4)
    B *= 2.0 ** 200                   # keeps the products of the subnormal row in the normal range
    A[5, :] = 0                       # zero row -> zero row of C
    B[:, 7] = 0
    A[9, 3] = np.inf                  # non-finite -> NaN row / column, nothing else disturbed
    B[11, 2] = np.nan
    A[20, :] *= 2.0 ** -1040          # subnormal row
    B[:, 30] *= 2.0 ** 700            # huge column
    C, st = run_z(A, B, 16)
    assert (C[5, np.arange(n) != 2] == 0).all() and (C[np.arange(m) != 9, 7] == 0).all()
    assert np.isnan(C[9, :]).all() and np.isnan(C[:, 2]).all()
    ok_r = np.array([i for i in range(m) if i != 9])
    ok_c = np.array([j for j in range(n) if j != 2])
    A2, B2 = A[ok_r, :], B[:, ok_c]
    Cref, D = direct.zgemm4m_dd(A2, B2)
    assert direct.componentwise_error(C[np.ix_(ok_r, ok_c)], Cref, D) <= TOL_Z
    ref = staged.zgemm2m_staged(A2, B2, 16, upto="pre")
    assert (st["eA"][ok_r] == ref["eA"]).all() and (st["eB"][ok_c] == ref["eB"]).all()


def test_empty_dimensions():
    A, B = inputs.complex_inputs(6, 5, 4, seed=5)
    with Workspace(4096):
        C = empty_dev(6, 5, torch.complex128, fill=9.0)
        b.zgemm2m(to_dev(A)[:, :0], to_dev(B)[:0, :], C, 16)        # k = 0: C = 0
        assert (to_host(C) == 0).all()
        b.zgemm2m(to_dev(A)[:0, :], to_dev(B), empty_dev(0, 5, torch.complex128), 16)   # m = 0: no-op
        b.zherk2m(to_dev(A)[:0, :], empty_dev(0, 0, torch.complex128), 16)
        b.device_status()


def test_workspace_too_small_is_refused():
    A, B = inputs.complex_inputs(64, 64, 64, seed=5)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, 64, 64, 64, 16) - 256):
        with pytest.raises(b.Gemm2mError, match="WORKSPACE"):
            b.zgemm2m(to_dev(A), to_dev(B), empty_dev(64, 64, torch.complex128), 16)
    b.set_workspace(None)
    with pytest.raises(b.Gemm2mError, match="WORKSPACE"):
        b.zgemm2m(to_dev(A), to_dev(B), empty_dev(64, 64, torch.complex128), 16)


@pytest.mark.parametrize("shape,nmod", [((100, 90, 150), 7), ((257, 300, 1000), 7), ((64, 64, 64), 22), ((128, 128, 256), 9)])
def test_cgemm_parity(shape, nmod):
    m, n, k = shape
    A, B = inputs.complex_inputs(m, n, k, seed=8, dtype=np.complex64)
    C, st = run_z(A, B, nmod, cplx=torch.complex64)
    assert C.dtype == np.complex64
    ref = staged.zgemm2m_staged(A, B, nmod, out_bits=24)
    assert (st["eA"] == ref["eA"]).all() and (st["eB"] == ref["eB"]).all()
    for j in range(nmod):
        for sgn in range(2):
            assert (st["Apm"][sgn, j, :, :k] == ref["Apm"][j][sgn]).all()
            assert (st["Cpm"][sgn, j, :, :m] == ref["Cpm"][j][sgn].T).all()
    Cref, D = direct.zgemm4m_dd(A, B)
    assert direct.componentwise_error(C, Cref, D) <= TOL_C
    # double rounding (53 then 24 bits) may differ from the single rounding by one float ulp
    spacing = np.spacing(np.abs(ref["C"].real).astype(np.float32)).astype(np.float64)
    assert (np.abs(C.real.astype(np.float64) - ref["C"].real) <= spacing).all()


@pytest.mark.parametrize("n,k,nmod", [(96, 200, 16), (257, 129, 16), (130, 300, 17), (64, 64, 21), (70, 50, 7), (33, 40, 8), (20, 10, 1)])
def test_zherk_parity(n, k, nmod):
    A = inputs.herk_input(n, k, seed=9)
    with Workspace(max(b.workspace_bytes(b.OP_ZHERK, n, n, k, nmod), b.workspace_bytes(b.OP_ZGEMM, n, n, k, nmod))) as ws:
        C = empty_dev(n, n, torch.complex128, fill=-5.0)
        b.zherk2m(to_dev(A), C, nmod)
        b.device_status()
        st = ws.stages(b.OP_ZHERK, n, n, k, nmod)
        Ch = to_host(C)
        Cg = empty_dev(n, n, torch.complex128)
        b.zgemm2m(to_dev(A), to_dev(np.asfortranarray(A.conj().T)), Cg, nmod)
        b.device_status()
        Cg = to_host(Cg)
    ref = staged.zgemm2m_staged(A, np.asfortranarray(A.conj().T), nmod, herk=True)
    assert (st["eA"] == ref["eA"]).all()
    for j in range(nmod):
        assert (st["Cpm"][0, j, :, :n] == ref["Cpm"][j][0].T).all()          # C+ = A+ A-^T (Section 5)
    low = np.tril(np.ones((n, n), dtype=bool))
    assert (Ch[~low] == -5.0).all()                                           # strict upper triangle untouched
    assert (np.diag(Ch).imag == 0).all()
    Cref, D = direct.zgemm4m_dd(A, np.asfortranarray(A.conj().T))
    if nmod >= 16:                                                            # fewer moduli: the error bound is that of their M; the stages are still exact
        assert direct.componentwise_error(Ch[low], Cref[low], D[low]) <= TOL_Z
    assert ulp_distance(Ch[low].real, ref["C"][low].real).max() <= 1 and ulp_distance(Ch[low].imag, ref["C"][low].imag).max() <= 1
    if ref["Pt"] % 2 == 0:                                                    # same scale split: identical integers, identical bits
        assert (Ch[low] == Cg[low]).all()


def test_device_status_and_launch_counts():
    A, B = inputs.complex_inputs(256, 256, 256, seed=2)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, 256, 256, 256, 16)):
        b.set_profiling(True)
        try:
            b.zgemm2m(to_dev(A), to_dev(B), empty_dev(256, 256, torch.complex128), 16)
            b.device_status()
            ms, calls = b.phase_ms()
            total, per = b.last_launch_count()
        finally:
            b.set_profiling(False)
    assert calls == 1 and all(x >= 0 for x in ms) and sum(ms) > 0
    assert per == [2, 2, 1, 2] and total == 7             # two scans, two residue launches, one GEMM launch, the post-processing's operand and its launch


def test_chained_launches_are_bitwise_identical_to_plain_ones_in_a_stream_of_calls():
    # The residue, GEMM and post-processing kernels are launched as programmatic dependents: a kernel may be resident before
    # the one in front of it has finished, and must not touch memory until it has.  Calls on different operands, sharing one
    # workspace, are enqueued back to back without a synchronisation in between; a kernel that read planes, exponents or C
    # early would pick up the previous call's.
    shapes = [(300, 200, 260), (129, 1100, 96), (520, 130, 1030)]
    ops = [inputs.complex_inputs(m, n, k, seed=40 + i, dist="phi", phi=1.0) for i, (m, n, k) in enumerate(shapes)]
    H = inputs.complex_inputs(260, 1, 300, seed=44)[0]
    dev = [(to_dev(A), to_dev(B)) for A, B in ops]
    dH = to_dev(H)
    need = max([b.workspace_bytes(b.OP_ZGEMM, m, n, k, 16) for m, n, k in shapes] + [b.workspace_bytes(b.OP_ZHERK, 260, 260, 300, 16)])
    results = {}
    with Workspace(need):
        for chained in (False, True):
            b.debug_set_chained_launch(chained)
            outs = []
            for rep in range(6):
                for (m, n, k), (dA, dB) in zip(shapes, dev):
                    C = empty_dev(m, n, torch.complex128, fill=float(rep))
                    b.zgemm2m(dA, dB, C, 16 if rep % 2 == 0 else 12)
                    outs.append(C)
                Ch = empty_dev(260, 260, torch.complex128, fill=1.0)
                b.zherk2m(dH, Ch, 16)
                outs.append(Ch)
            b.device_status()
            results[chained] = [to_host(C) for C in outs]
    for x, y in zip(results[False], results[True]):
        assert (x == y).all()
    ref = staged.zgemm2m_staged(ops[0][0], ops[0][1], 16)["C"]
    assert (results[True][0] == ref).mean() > 0.999


def test_panel_pipeline_is_bitwise_identical_and_joins_the_callers_stream():
    # zgemm2m cuts C into column panels; with the overlap switched on it post-processes them on an internal stream.  The result
    # must depend neither on the number of panels nor on the mode, and work queued on the caller's stream right after the call
    # must see all of C.
    m, n, k = 300, 2304, 256                      # 2304 columns -> 2 panels of 1280 / 1024
    A, B = inputs.complex_inputs(m, n, k, seed=17, dist="phi", phi=1.0)
    dA, dB = to_dev(A), to_dev(B)
    outs = []
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, 16)):
        side = torch.cuda.Stream()
        for panels, overlap in ((1, False), (4, True), (2, False), (4, False), (2, True)):
            b.debug_set_panels(panels)
            b.debug_set_overlap(overlap)
            C = empty_dev(m, n, torch.complex128, fill=7.0)
            snap = torch.empty_like(C)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                b.zgemm2m(dA, dB, C, 16, side)
                snap.copy_(C)                     # same stream, no synchronisation in between
            side.synchronize()
            b.device_status(side)
            outs.append((to_host(C), to_host(snap)))
        b.debug_set_panels(8)
    ref = staged.zgemm2m_staged(A, B, 16)["C"]
    for C, snap in outs:
        assert (C == outs[0][0]).all() and (snap == C).all()
    assert ulp_distance(outs[0][0].real, ref.real).max() <= 1 and ulp_distance(outs[0][0].imag, ref.imag).max() <= 1


def test_wide_c_in_more_than_four_panels():
    m, n, k = 70, 10368, 128                      # 10368 columns -> 5 panels of 2304 / 2048 / ... / 1152 columns
    A, B = inputs.complex_inputs(m, n, k, seed=19)
    dA, dB = to_dev(A), to_dev(B)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, 16)):
        outs = []
        for panels in (8, 1):
            b.debug_set_panels(panels)
            C = empty_dev(m, n, torch.complex128, fill=7.0)
            b.zgemm2m(dA, dB, C, 16)
            b.device_status()
            outs.append(to_host(C))
            if panels == 8:
                assert b.last_launch_count()[1][2] == 5          # one GEMM launch per panel
    assert (outs[0] == outs[1]).all()
    Cref, D = direct.zgemm4m_dd(A, B)
    assert direct.componentwise_error(outs[0], Cref, D) <= TOL_Z


def test_back_to_back_calls_of_different_sizes_share_a_workspace():
    shapes = [(512, 2048, 128), (100, 130, 200), (256, 4096, 64), (64, 1100, 300)]
    need = max(b.workspace_bytes(b.OP_ZGEMM, m, n, k, 16) for m, n, k in shapes)
    data = [inputs.complex_inputs(m, n, k, seed=20 + i) for i, (m, n, k) in enumerate(shapes)]
    with Workspace(need):
        dev = [(to_dev(A), to_dev(B), empty_dev(A.shape[0], B.shape[1], torch.complex128)) for A, B in data]
        for _ in range(2):
            for dA, dB, dC in dev:                # no synchronisation between the calls
                b.zgemm2m(dA, dB, dC, 16)
        b.device_status()
        got = [to_host(dC) for _, _, dC in dev]
    for (A, B), C in zip(data, got):
        Cref, D = direct.zgemm4m_dd(A, B)
        assert direct.componentwise_error(C, Cref, D) <= TOL_Z

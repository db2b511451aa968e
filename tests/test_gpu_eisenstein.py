"""GPU parity of the Eisenstein-integer variant (Sections 3.2, 4) against its CPU oracle, stage by stage.

The oracle works in the ring's basis {1, w} with the homomorphisms w -> s, s^2; the library holds an entry as
(u + v sqrt(-3))/2 and its planes are u +- (2s + 1) v = 2 (a + s b), 2 (a + s^2 b): twice the oracle's residues, and four times
its products.  Scale exponents, lattice points (through the planes), products and the lifted result are compared exactly."""
import numpy as np
import pytest
import torch

from oracle import direct, eisenstein as E, staged
from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host, ulp_distance  # noqa: E402

OP = b.OP_ZGEMM_EISENSTEIN


@pytest.fixture(autouse=True)
def _default_kernel():
    b.debug_set_gemm_kernel(0)
    b.debug_set_panels(8)
    yield
    b.debug_set_gemm_kernel(0)
    b.debug_set_panels(8)


def run_e(A, B, nmod, kernel=0):
    m, k = A.shape
    n = B.shape[1]
    b.debug_set_gemm_kernel(kernel)
    with Workspace(b.workspace_bytes(OP, m, n, k, nmod)) as ws:
        C = empty_dev(m, n, torch.complex128)
        b.zgemm2m_eisenstein(to_dev(A), to_dev(B), C, nmod)
        b.device_status()
        return to_host(C), ws.stages(OP, m, n, k, nmod)


@pytest.mark.parametrize("kernel", [1, 0], ids=["checkgemm", "tcgen05"])
@pytest.mark.parametrize("shape,nmod,dist,phi", [((200, 150, 300), 16, "phi", 1.0), ((129, 257, 128), 15, "uniform", 0.5),
                                                 ((64, 64, 64), 3, "uniform", 0.5), ((33, 19, 50), 23, "phi", 4.0),
                                                 ((40, 40, 520), 20, "uniform", 0.5), ((70, 90, 200), 8, "phi", 2.0)])
def test_every_stage_against_the_oracle(shape, nmod, dist, phi, kernel):
    m, n, k = shape
    A, B = inputs.complex_inputs(m, n, k, seed=11, dist=dist, phi=phi)
    C, st = run_e(A, B, nmod, kernel)
    ref = E.zgemm_eisenstein_staged(A, B, nmod)
    assert (st["eA"] == ref["eA"]).all() and (st["eB"] == ref["eB"]).all()
    for j, mj in enumerate(ref["moduli"]):
        for sgn in range(2):
            assert (st["Apm"][sgn, j, :, :k] == staged.sym(2 * ref["Apm"][j][sgn], mj)).all(), ("Apm", sgn, j)
            assert (st["Bpm"][sgn, j, :, :k] == staged.sym(2 * ref["Bpm"][j][sgn].T, mj)).all(), ("Bpm", sgn, j)
            assert (st["Apm"][sgn, j, :, k:] == 0).all() and (st["Bpm"][sgn, j, :, k:] == 0).all()
            assert (st["Cpm"][sgn, j, :, :m] == staged.sym(4 * ref["Cpm"][j][sgn].T, mj)).all(), ("Cpm", sgn, j)
    # the real part U/2 is rounded once from an exact integer; the imaginary part carries the double-double factor sqrt(3)/2
    assert ulp_distance(C.real, ref["C"].real).max() <= 1 and ulp_distance(C.imag, ref["C"].imag).max() <= 1
    assert (C.real == ref["C"].real).mean() > 0.999 and (C.imag == ref["C"].imag).mean() > 0.99
    Cref, D = direct.zgemm4m_dd(A, B)
    if nmod >= 16:
        assert direct.componentwise_error(C, Cref, D) <= 1e-14


def test_lattice_rounding_on_cell_boundaries_and_special_values():
    # one row per scale; the first entry of a row fixes its exponent e so that the other entries are the listed values in
    # lattice units: lattice points, deep holes (three nearest points), edge midpoints (two), tiny and subnormal numbers
    rt3 = np.sqrt(3.0)
    vals = [0.0, 1.0, -0.5 + 0.5j * rt3, 0.5 + 0.5j / rt3, 0.5, 0.25 + 0.25j * rt3, -0.5 - 0.5j / rt3, 1e-300, -1e-300j,
            0.499999 + 0.2886j, 3.5 + 2.5j * rt3, -7.25 + 0.01j, 5e-324, 2.0 ** -40 * (1 + 1j), 1.5, 2.5 - 1.5j * rt3,
            1.0 + 1j / rt3, 1000.5 + 1000.5j / rt3, 0.5 + 0.8660254037844386j, 0.5 + 0.8660254037844387j]
    k = len(vals) + 1
    B = np.eye(k, 4, dtype=np.complex128)
    for nmod in (6, 16):
        M = staged.product(E.greedy_eisenstein_moduli()[:nmod])
        Pt, PA, PB, ck = E.scaling_targets_e(M, k)
        sigmas = (0, 20, -30, -1005, 900)         # the last two: exponents outside the kernel's fast scaling path
        A = np.zeros((len(sigmas), k), dtype=np.complex128)
        for i, sg in enumerate(sigmas):
            A[i, 0] = 1.5 * 2.0 ** (sg + PA - ck - 1)
            A[i, 1:] = np.array(vals) * 2.0 ** sg
        C, st = run_e(A, B, nmod, kernel=1)
        ref = E.zgemm_eisenstein_staged(A, B, nmod)
        assert list(ref["eA"]) == list(sigmas) and (st["eA"] == ref["eA"]).all()
        assert ref["Aq"][1][0, 3] == 1 and ref["Aq"][0][0, 3] == 0          # w itself is a lattice point: (a, b) = (0, 1)
        for j, mj in enumerate(ref["moduli"]):
            for sgn in range(2):
                assert (st["Apm"][sgn, j, :, :k] == staged.sym(2 * ref["Apm"][j][sgn], mj)).all(), (nmod, sgn, j)
        assert ulp_distance(C.real, ref["C"].real).max() <= 1 and ulp_distance(C.imag, ref["C"].imag).max() <= 1


def test_transposes_alpha_beta_and_padding():
    m, n, k, nmod = 70, 45, 130, 16
    A, B = inputs.complex_inputs(m, n, k, seed=5, dist="phi", phi=1.0)
    rng = np.random.default_rng(1)
    C0 = rng.standard_normal((m, n)) + 1j * rng.standard_normal((m, n))
    alpha, beta = 0.75 - 0.5j, -1.25 + 2j
    with Workspace(b.workspace_bytes(OP, m, n, k, nmod)):
        for ta, tb in (("N", "N"), ("C", "T"), ("T", "C")):
            As = A if ta == "N" else (A.T if ta == "T" else A.conj().T)      # stored so that op(stored) = A
            Bs = B if tb == "N" else (B.T if tb == "T" else B.conj().T)
            Cf = empty_dev(96, n, torch.complex128, fill=-7)
            Cf[:m] = to_dev(C0)
            b.zgemm2m_eisenstein_ex(ta, tb, alpha, to_dev(As), to_dev(Bs), beta, Cf[:m], nmod)
            b.device_status()
            C = to_host(Cf)
            assert (C[m:] == -7).all()
            ref, D = direct.zgemm_ex_dd(ta, tb, alpha, As, Bs, beta, C0)
            assert np.max(np.abs(C[:m] - ref) / D) < 1e-14, (ta, tb)


def test_more_bits_than_the_gaussian_set_and_error_paths():
    # 23 Eisenstein moduli carry M = 2^160.9 against 2^152 for the 22 Gaussian ones: on inputs with a wide exponent span the
    # variant is at least as accurate as zgemm2m with all 22 2M moduli
    m, n, k = 48, 40, 160
    A, B = inputs.complex_inputs(m, n, k, seed=3, dist="phi", phi=6.0)
    Cref, D = direct.zgemm4m_dd(A, B)
    Ce, _ = run_e(A, B, 23)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, 22)):
        Cg = empty_dev(m, n, torch.complex128)
        b.zgemm2m(to_dev(A), to_dev(B), Cg, 22)
        Cg = to_host(Cg)
    err_e, err_g = direct.componentwise_error(Ce, Cref, D), direct.componentwise_error(Cg, Cref, D)
    ref = E.zgemm_eisenstein_staged(A, B, 23)
    assert err_e <= 1.01 * direct.componentwise_error(ref["C"], Cref, D) + 1e-16
    assert err_e < err_g
    with Workspace(1 << 20):
        C = empty_dev(8, 8, torch.complex128)
        X = to_dev(np.ones((8, 8), dtype=np.complex128))
        with pytest.raises(b.Gemm2mError):
            b.zgemm2m_eisenstein(X, X, C, 24)               # only 23 moduli
        with pytest.raises(b.Gemm2mError):
            b.zgemm2m_eisenstein(X, X, C, 1)                # P_B - c_k < 2: too few moduli for the lattice rounding


def test_2048_sampled_against_the_oracle():
    m = n = k = 2048
    nmod = 16
    A, B = inputs.complex_inputs(m, n, k, seed=2, dist="phi", phi=0.5)
    C, st = run_e(A, B, nmod)
    rng = np.random.default_rng(0)
    rows, cols = rng.integers(0, m, 24), rng.integers(0, n, 24)
    ref = E.zgemm_eisenstein_staged(A[rows], B[:, cols], nmod, upto="quantise")
    full_eA = staged.scaling_exponents(A, 1, ref["PA"], ref["ck"])
    full_eB = staged.scaling_exponents(B, 0, ref["PB"], ref["ck"])
    assert (st["eA"] == full_eA).all() and (st["eB"] == full_eB).all()
    sub = E.zgemm_eisenstein_staged(A[rows], B[:, cols], nmod)
    assert ulp_distance(C[np.ix_(rows, cols)].real, sub["C"].real).max() <= 1
    assert ulp_distance(C[np.ix_(rows, cols)].imag, sub["C"].imag).max() <= 1
    Cref, D = direct.zgemm4m_dd_samples(A, B, np.stack([rows, cols], axis=1))
    assert np.max(np.abs(C[rows, cols] - Cref) / D) < 1e-14


def test_error_and_time_against_modulus_count_beside_the_gaussian_set():
    """4096^3, phi = 0.5: the error of the Eisenstein variant falls by about M^-1/2 per modulus (Section 3.1) down to the
    rounding floor; per modulus it is at least as accurate as zgemm2m from the point where its M is larger (Section 4: the
    Eisenstein set decreases more slowly).  The table itself is printed as one JSON line (`pytest -s` or `-rP` shows it)."""
    import json
    import math
    m = n = k = 4096
    A, B = inputs.complex_inputs(m, n, k, seed=2, dist="phi", phi=0.5)
    pairs = inputs.sample_indices(m, n, 1024, seed=7, tile=128)
    Cs, Ds = direct.zgemm4m_dd_samples(A, B, pairs)
    idx = torch.from_numpy(pairs).cuda()
    dA, dB = to_dev(A), to_dev(B)
    nmods = list(range(8, 24))
    rows = []
    with Workspace(max(b.workspace_bytes(OP, m, n, k, 23), b.workspace_bytes(b.OP_ZGEMM, m, n, k, 22))):
        C = empty_dev(m, n, torch.complex128)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for nmod in nmods:
            row = dict(nmod=nmod)
            for name, fn, mods in (("eis", b.zgemm2m_eisenstein, E.greedy_eisenstein_moduli()),
                                   ("gauss", b.zgemm2m, staged.greedy_2m_moduli())):
                if nmod > len(mods):
                    continue
                fn(dA, dB, C, nmod)                  # warm
                e0.record()
                for _ in range(3):
                    fn(dA, dB, C, nmod)
                e1.record()
                b.device_status()
                got = C[idx[:, 0], idx[:, 1]].cpu().numpy()
                row[name] = dict(log2M=round(math.log2(staged.product(mods[:nmod])), 2), ms=e0.elapsed_time(e1) / 3,
                                 max_err=direct.componentwise_error(got, Cs, Ds))
            rows.append(row)
    errs = {r["nmod"]: r["eis"]["max_err"] for r in rows}
    floor = 4e-16
    for a, c in zip(nmods, nmods[1:]):
        assert errs[c] <= max(1.5 * errs[a], floor), (a, c, errs)
        if errs[c] > 20 * floor:
            assert errs[c] < errs[a] / 3, (a, c, errs)
    assert errs[16] <= 1e-14 and all(errs[nm] <= 4 * floor for nm in nmods if nm >= 18)
    slope = math.log2(errs[8] / errs[12]) / (rows[4]["eis"]["log2M"] - rows[0]["eis"]["log2M"])
    assert 0.35 < slope < 0.65, slope
    for r in rows:                                   # same error law for both rings: compare at equal M, not at equal N
        if "gauss" in r and r["eis"]["max_err"] > 20 * floor and r["gauss"]["max_err"] > 20 * floor:
            ratio = math.log2(r["gauss"]["max_err"] / r["eis"]["max_err"])
            gap = 0.5 * (r["eis"]["log2M"] - r["gauss"]["log2M"])
            assert abs(ratio - gap) < 2.5, (r, ratio, gap)
    print(json.dumps(rows))


def test_k_beyond_the_int32_range_of_one_gemm_and_ragged_padded_operands():
    # k above 2^31 / 123^2 = 141 944: the GEMM runs in two K chunks whose residues are added modulo m_j
    m, n, k, nmod = 3, 2, 142200, 4
    A, B = inputs.complex_inputs(m, n, k, seed=9, dist="uniform")
    C, st = run_e(A, B, nmod)
    ref = E.zgemm_eisenstein_staged(A, B, nmod)
    for j, mj in enumerate(ref["moduli"]):
        for sgn in range(2):
            assert (st["Cpm"][sgn, j, :, :m] == staged.sym(4 * ref["Cpm"][j][sgn].T, mj)).all(), (sgn, j)
    assert ulp_distance(C.real, ref["C"].real).max() <= 1 and ulp_distance(C.imag, ref["C"].imag).max() <= 1
    # ragged sizes with padded leading dimensions; the padding of C stays untouched
    m, n, k, nmod = 131, 77, 301, 21
    A, B = inputs.complex_inputs(m, n, k, seed=10, dist="phi", phi=2.0)
    pad = lambda a, ld: np.asfortranarray(np.vstack([a, np.full((ld - a.shape[0], a.shape[1]), 99 + 1j, dtype=a.dtype)]))
    with Workspace(b.workspace_bytes(OP, m, n, k, nmod)):
        Cf = empty_dev(140, n, torch.complex128, fill=-7)
        b.zgemm2m_eisenstein(to_dev(pad(A, 136))[:m], to_dev(pad(B, 320))[:k], Cf[:m], nmod)
        b.device_status()
        Cf = to_host(Cf)
    ref = E.zgemm_eisenstein_staged(A, B, nmod)
    assert (Cf[m:] == -7).all()
    assert ulp_distance(Cf[:m].real, ref["C"].real).max() <= 1 and ulp_distance(Cf[:m].imag, ref["C"].imag).max() <= 1

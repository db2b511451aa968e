"""Pins for the CPU oracle: values the paper prints, closed forms, brute force, library routines.

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong sign, a
transposed operand, a wrong constant) fails it.  None of these needs a GPU.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import direct, staged
from paper_2609_05419_b200 import inputs
from conftest import read_golden


@pytest.fixture(scope="module")
def printed(golden_dir):
    return read_golden(os.path.join(golden_dir, "moduli_printed.txt"))


# ------------------------------------------------------------------ constants
def test_moduli_match_printed_list(printed):
    mods = staged.greedy_2m_moduli()
    assert mods[:14] == printed["m2m_prefix"]
    assert mods[-2:] == printed["m2m_suffix"]
    assert len(mods) == 22
    assert round(math.log2(staged.product(mods[:16])) - 0.5) == printed["m2m_log2_first16"][0]   # 2^117.69
    assert round(math.log2(staged.product(mods))) == printed["m2m_log2_all"][0]                  # 2^152.08
    for a in mods:
        for b in mods:
            assert a == b or math.gcd(a, b) == 1


def test_greedy_reading_reproduces_real_modulus_set(printed):
    # the same greedy walk without the 2M filter must give the paper's real-Ozaki-II list
    kept = []
    for cand in range(256, 1, -1):
        if all(math.gcd(cand, q) == 1 for q in kept):
            kept.append(cand)
    assert kept[:10] == printed["mreal_prefix"]
    n117 = printed["mreal_count_for_117"][0]
    assert 117 <= math.log2(staged.product(kept[:n117])) < 118
    assert round(math.log2(staged.product(kept))) == printed["mreal_log2_all"][0]


def test_2m_modulus_criterion_by_brute_force():
    # Section 2: s with s^2 = -1 (mod m) exists iff m is a product of primes = 1 (mod 4), m odd
    for m in range(3, 258, 2):
        exists = any((s * s + 1) % m == 0 for s in range(m))
        assert exists == staged.is_2m_modulus(m), m


def test_roots_two_derivations():
    for m in staged.greedy_2m_moduli():
        s = staged.sqrt_minus_one(m)
        assert (s * s) % m == m - 1
        assert (2 * staged.inv2(m)) % m == 1
        # Section 2.1: m = u^2 + v^2 with gcd(u, v) = 1 and s = -u v^-1 (mod m), up to sign / choice of root
        found = False
        for u in range(1, 16):
            v2 = m - u * u
            v = math.isqrt(v2) if v2 > 0 else 0
            if v > 0 and v * v == v2 and math.gcd(u, v) == 1:
                cand = (-u * pow(v, -1, m)) % m
                assert (cand * cand) % m == m - 1
                found = found or cand in (s, m - s)
        assert found, m
    assert staged.sqrt_minus_one(241) == 64 and (-15 * pow(4, -1, 241)) % 241 == 241 - 64


def test_2m_identity_brute_force():
    # (2c) applied to (2b) of (2a) equals the complex product mod m, for every small Gaussian integer pair
    rng = range(-3, 4)
    for m in staged.greedy_2m_moduli():
        s = staged.sqrt_minus_one(m)
        for ar in rng:
            for ai in rng:
                ap, am = staged.pre_2m(ar, ai, m, s)
                for br in rng:
                    for bi in rng:
                        bp, bm = staged.pre_2m(br, bi, m, s)
                        cp, cm = staged.sym(ap * bp, m), staged.sym(am * bm, m)
                        # (2b): C+- = (ArBr - AiBi) +- s (ArBi + AiBr)
                        assert (cp - ((ar * br - ai * bi) + s * (ar * bi + ai * br))) % m == 0
                        assert (cm - ((ar * br - ai * bi) - s * (ar * bi + ai * br))) % m == 0
                        cr, ci = staged.post_2m(cp, cm, m, s)
                        assert (cr - (ar * br - ai * bi)) % m == 0
                        assert (ci - (ar * bi + ai * br)) % m == 0
                        assert abs(cr) <= (m - 1) // 2 and abs(ci) <= (m - 1) // 2


def test_2m_hand_example():
    # m = 241, s = 64, a = 3 + 2i, b = 1 - 4i, ab = 11 - 10i, worked through (2a)-(2c) by hand
    m, s = 241, 64
    ap, am = staged.pre_2m(3, 2, m, s)
    bp, bm = staged.pre_2m(1, -4, m, s)
    assert (ap % m, am % m, bp % m, bm % m) == (131, 116, 227, 16)
    cp, cm = (ap * bp) % m, (am * bm) % m
    assert (cp, cm) == (94, 169)
    assert staged.inv2(m) == 121
    assert staged.post_2m(cp, cm, m, s) == (11, -10)


def test_crt_roundtrip_known_integers():
    rng = np.random.default_rng(5)
    for nmod in (1, 2, 3, 8, 16, 22):
        mods = staged.greedy_2m_moduli()[:nmod]
        M = staged.product(mods)
        h = (M - 1) // 2
        for x in [0, 1, -1, h, -h, h - 1] + [int(rng.integers(-2 ** 62, 2 ** 62)) % M - h for _ in range(20)]:
            res = [staged.sym(x, q) for q in mods]
            assert staged.lift(staged.crt(res, mods), M) == staged.lift(x, M)
        # one step beyond the range wraps around, as the definition says
        assert staged.lift(staged.crt([staged.sym(h + 1, q) for q in mods], mods), M) == -h


# ------------------------------------------------------------------ O-int
@pytest.mark.parametrize("shape", [(1, 1, 1), (2, 3, 1), (3, 2, 5), (7, 5, 3), (4, 4, 9)])
def test_int128_product_vs_python_ints(shape):
    m, n, k = shape
    rng = np.random.default_rng(11 + m * n * k)
    big = 2 ** 55
    Ar, Ai = rng.integers(-big, big, size=(m, k)), rng.integers(-big, big, size=(m, k))
    Br, Bi = rng.integers(-big, big, size=(k, n)), rng.integers(-big, big, size=(k, n))
    cr, ci = direct.gauss4m_exact(Ar, Ai, Br, Bi)
    pr, pi = direct.gauss4m_python(Ar, Ai, Br, Bi)
    assert (cr == pr).all() and (ci == pi).all()


def test_int128_product_vs_numpy_complex_matmul():
    # int8-range data: numpy's complex matmul is exact here (all values far below 2^53)
    Ar, Ai, Br, Bi = inputs.gaussian_int_inputs(33, 17, 70, seed=3)
    cr, ci = direct.gauss4m_exact(Ar, Ai, Br, Bi)
    Z = (Ar.astype(np.float64) + 1j * Ai) @ (Br.astype(np.float64) + 1j * Bi)
    assert (cr.astype(np.float64) == Z.real).all() and (ci.astype(np.float64) == Z.imag).all()
    # asymmetric shapes catch a transposed operand; the scalar case pins the sign convention i^2 = -1
    cr1, ci1 = direct.gauss4m_exact([[3]], [[2]], [[1]], [[-4]])
    assert (int(cr1[0, 0]), int(ci1[0, 0])) == (11, -10)


def test_symmetric_residue_definition():
    M = 241 * 233
    h = (M - 1) // 2
    for x in range(-3 * M, 3 * M, 997):
        r = direct.symmetric_residue(x, M)
        assert -h <= r <= h and (r - x) % M == 0


# ------------------------------------------------------------------ O-fp
def test_dd_product_vs_exact_rationals():
    A, B = inputs.complex_inputs(3, 4, 6, seed=2, dist="phi", phi=2.0)
    C, D = direct.zgemm4m_dd(A, B)
    for i in range(3):
        for j in range(4):
            er = sum(Fraction(A[i, p].real) * Fraction(B[p, j].real) - Fraction(A[i, p].imag) * Fraction(B[p, j].imag) for p in range(6))
            ei = sum(Fraction(A[i, p].real) * Fraction(B[p, j].imag) + Fraction(A[i, p].imag) * Fraction(B[p, j].real) for p in range(6))
            d = sum(abs(A[i, p]) * abs(B[p, j]) for p in range(6))
            # correctly rounded up to the last bit of the larger product (double-double carries 100+ bits)
            assert abs(Fraction(C[i, j].real) - er) <= Fraction(d) * Fraction(1, 2 ** 52)
            assert abs(Fraction(C[i, j].imag) - ei) <= Fraction(d) * Fraction(1, 2 ** 52)
            assert abs(D[i, j] - d) <= 1e-15 * d


def test_dd_product_recovers_cancellation():
    # ar*br - ai*bi with massive cancellation: plain double loses everything, double-double must not
    a = np.array([[(1 + 2.0 ** -30) + 1j * (1 - 2.0 ** -30)]], order="F")
    b = np.array([[(1 + 2.0 ** -30) + 1j * (1 + 2.0 ** -30)]], order="F")
    C, _ = direct.zgemm4m_dd(a, b)
    exact_r = Fraction(a[0, 0].real) * Fraction(b[0, 0].real) - Fraction(a[0, 0].imag) * Fraction(b[0, 0].imag)
    assert Fraction(C[0, 0].real) == exact_r        # exactly representable: 2^-29 + 2^-59 ... fits a double


def test_dd_product_equals_integer_product_on_integer_data():
    Ar, Ai, Br, Bi = inputs.gaussian_int_inputs(20, 31, 45, seed=8)
    A = np.asfortranarray(Ar.astype(np.float64) + 1j * Ai)
    B = np.asfortranarray(Br.astype(np.float64) + 1j * Bi)
    C, D = direct.zgemm4m_dd(A, B)
    cr, ci = direct.gauss4m_exact(Ar, Ai, Br, Bi)
    assert (C.real == cr.astype(np.float64)).all() and (C.imag == ci.astype(np.float64)).all()
    assert np.allclose(D, np.abs(A) @ np.abs(B), rtol=1e-13)


def test_dd_product_vs_library_matmul_and_samples():
    A, B = inputs.complex_inputs(40, 23, 64, seed=4)
    C, D = direct.zgemm4m_dd(A, B)
    assert direct.componentwise_error(A @ B, C, D) < 64 * 2.3e-16
    pairs = inputs.sample_indices(40, 23, 50, seed=1, tile=16)
    Cs, Ds = direct.zgemm4m_dd_samples(A, B, pairs)
    assert (Cs == C[pairs[:, 0], pairs[:, 1]]).all() and (Ds == D[pairs[:, 0], pairs[:, 1]]).all()


# ------------------------------------------------------------------ staged Algorithm 1
@pytest.mark.parametrize("nmod", [1, 2, 3, 8])
def test_staged_integer_path_equals_4m_definition(nmod):
    # Section 6: the multiplication method (2M vs 4M) cannot change the integer result
    Ar, Ai, Br, Bi = inputs.gaussian_int_inputs(24, 19, 37, seed=nmod)
    st = staged.gemm2m_int_staged(Ar, Ai, Br, Bi, nmod)
    er, ei = direct.gauss4m_mod(Ar, Ai, Br, Bi, st["M"])
    assert (st["Xr"].astype(np.int64) == er).all() and (st["Xi"].astype(np.int64) == ei).all()
    if nmod == 3:        # |c| <= 2*37*16^2 < M/2: no wrap, equals the exact product
        cr, ci = direct.gauss4m_exact(Ar, Ai, Br, Bi)
        assert (st["Xr"] == cr).all() and (st["Xi"] == ci).all()
    if nmod == 1:        # M = 241 wraps for sure
        cr, _ = direct.gauss4m_exact(Ar, Ai, Br, Bi)
        assert (st["Xr"] != cr).any()


def test_scaling_rule_and_truncation_invariants():
    A, B = inputs.complex_inputs(17, 13, 300, seed=6, dist="phi", phi=2.0)
    A[3, :] = 0                                   # zero row: exponent 0, quantises to zero
    for nmod in (3, 7, 16, 22):
        st = staged.zgemm2m_staged(A, B, nmod, upto="pre")
        assert st["eA"][3] == 0
        for (qr, qi), e, Z, axis, P in ((st["Aq"], st["eA"], A, 1, st["PA"]), (st["Bq"], st["eB"], B, 0, st["PB"])):
            eb = e[:, None] if axis == 1 else e[None, :]
            for q, part in ((qr, Z.real), (qi, Z.imag)):
                for idx in np.ndindex(q.shape):
                    exact = Fraction(float(part[idx])) / Fraction(2) ** int(np.broadcast_to(eb, q.shape)[idx])
                    assert abs(q[idx]) <= abs(exact) < abs(q[idx]) + 1        # truncation toward zero
                    assert (q[idx] >= 0) == (exact >= 0) or q[idx] == 0
            # the row/column 2-norm bound that makes |X| <= 2^Pt
            sq = (qr.astype(object) ** 2 + qi.astype(object) ** 2).sum(axis=axis)
            assert all(int(v) <= 4 ** P for v in sq)
        assert st["PA"] + st["PB"] == st["Pt"] and 2 ** st["Pt"] <= (st["M"] - 1) // 2 < 2 ** (st["Pt"] + 1)


def test_scaling_rule_wastes_less_than_one_bit_beyond_ck():
    # The largest part of a row quantises into [2^(P - c_k - 1), 2^(P - c_k)): the budget P is used up to the c_k bits the
    # sqrt(2k) factor of the 2-norm bound takes and less than one more.  An exponent one larger (a bit wasted per operand, which
    # the overflow bound and the error bound alone would not notice) fails the lower limit.
    rng = np.random.default_rng(8)
    for nmod, k in ((7, 64), (16, 300), (16, 8192), (22, 100)):
        vals = np.concatenate([2.0 ** rng.integers(-300, 300, 6), rng.uniform(1.0, 2.0, 6) * 2.0 ** rng.integers(-40, 40, 6),
                               [np.nextafter(2.0, 1.0), 5e-324, 1.7e308]])
        A = np.asfortranarray(np.repeat(vals[:, None], k, axis=1) * (1 + 0j))          # every entry of a row equals its maximum
        B = np.asfortranarray(np.repeat(vals[None, :], k, axis=0) * (0 + 1j))
        st = staged.zgemm2m_staged(A, B, nmod, upto="pre")
        ck = staged.scaling_targets(st["M"], k)[3]
        for q, P in ((st["Aq"][0][:, 0], st["PA"]), (st["Bq"][1][0, :], st["PB"])):
            lo, hi = P - ck - 1, P - ck
            assert all(2 ** lo <= int(v) < 2 ** hi for v in q if lo >= 0), (nmod, k)


@pytest.mark.parametrize("nmod", [14, 16, 22])
def test_staged_float_path_meets_error_bound_and_equals_4m_on_quantised(nmod):
    A, B = inputs.complex_inputs(12, 9, 100, seed=9, dist="phi", phi=0.5)
    st = staged.zgemm2m_staged(A, B, nmod)
    assert all(abs(int(v)) <= 2 ** st["Pt"] for v in st["Xr"].ravel())
    assert all(abs(int(v)) <= 2 ** st["Pt"] for v in st["Xi"].ravel())
    # the 2M route reproduces the plain integer product of the quantised matrices (no wrap by the bound)
    pairs = np.array([(i, j) for i in range(12) for j in range(9)])
    Xs, vals = staged.staged_samples(st, pairs)
    assert all(int(st["Xr"][i, j]) == xr and int(st["Xi"][i, j]) == xi for (i, j), (xr, xi) in zip(pairs.tolist(), Xs))
    assert (vals == st["C"][pairs[:, 0], pairs[:, 1]]).all()
    Cref, D = direct.zgemm4m_dd(A, B)
    err = direct.componentwise_error(st["C"], Cref, D)
    assert err <= (1e-13 if nmod == 14 else 1e-14)


def test_staged_error_falls_with_modulus_count():
    # Section 3.1: error ~ O(M^-1/2): each extra modulus (~2^7.5) buys about 2^3.7 until the rounding floor
    A, B = inputs.complex_inputs(10, 8, 64, seed=12)
    Cref, D = direct.zgemm4m_dd(A, B)
    errs = [direct.componentwise_error(staged.zgemm2m_staged(A, B, n)["C"], Cref, D) for n in (6, 8, 10, 12)]
    assert all(a > 20 * b for a, b in zip(errs, errs[1:])), errs
    M6, M12 = (staged.product(staged.greedy_2m_moduli()[:n]) for n in (6, 12))
    ratio = math.log2(errs[0] / errs[-1]) / math.log2(M12 / M6)
    assert 0.4 < ratio < 0.6, ratio


def test_staged_complex64_rounding():
    A, B = inputs.complex_inputs(9, 7, 50, seed=13, dtype=np.complex64)
    st = staged.zgemm2m_staged(A, B, 7, out_bits=24)
    C32 = st["C"].astype(np.complex64)
    assert (C32.astype(np.complex128) == st["C"]).all()          # already on the float32 grid
    Cref, D = direct.zgemm4m_dd(A, B)
    assert direct.componentwise_error(C32, Cref, D) <= 2e-6


def test_round_int_nearest_even_vs_python_float():
    rng = np.random.default_rng(3)
    xs = [int(rng.integers(-2 ** 62, 2 ** 62)) * int(rng.integers(1, 2 ** 60)) + int(rng.integers(-5, 5)) for _ in range(300)]
    xs += [2 ** 53 + 1, 2 ** 53 + 2, 2 ** 53 + 3, -(2 ** 54 + 2), 3 * 2 ** 52 + 0, (2 ** 53 - 1) * 2 ** 40 + 2 ** 39]
    for x in xs:
        y, t = staged.round_int_nearest_even(x, 53)
        assert math.ldexp(float(y), t) == float(x)               # Python's int -> float is round-half-even


def test_herk_symmetry_and_equivalence():
    A = inputs.herk_input(11, 40, seed=14)
    B = np.asfortranarray(A.conj().T)
    st = staged.zgemm2m_staged(A, B, 16, herk=True)
    assert st["Pt"] % 2 == 0
    for (Ap, Am), (Bp, Bm), (Cp, Cm) in zip(st["Apm"], st["Bpm"], st["Cpm"]):
        assert (Bp == Am.T).all() and (Bm == Ap.T).all()         # residues of A^H are the swapped planes, transposed
        assert (Cm == Cp.T).all()                                # Section 5: C- = C+^T
    assert (st["Xr"] == st["Xr"].T).all() and (st["Xi"] == -st["Xi"].T).all()
    assert all(int(v) == 0 for v in np.diag(st["Xi"]))
    st2 = staged.zgemm2m_staged(A, B, 16, herk=False)            # Pt even: same scaling, identical integers
    assert (st2["Xr"] == st["Xr"]).all() and (st2["Xi"] == st["Xi"]).all()


# ------------------------------------------------------------------ rank-k family (Section 5)
def test_two_product_dd_sum_vs_exact_rationals():
    rng = np.random.default_rng(21)
    mk = lambda r, c: np.asfortranarray(rng.standard_normal((r, c)) * np.exp(2 * rng.standard_normal((r, c))) +
                                        1j * rng.standard_normal((r, c)))
    A1, A2, B1, B2 = mk(3, 5), mk(3, 5), mk(5, 2), mk(5, 2)
    C, D = direct.zgemm4m_dd2(A1, B1, A2, B2)
    for i in range(3):
        for j in range(2):
            er = ei = Fraction(0)
            d = 0.0
            for A, B in ((A1, B1), (A2, B2)):
                for p in range(5):
                    ar, ai, br, bi = (Fraction(float(v)) for v in (A[i, p].real, A[i, p].imag, B[p, j].real, B[p, j].imag))
                    er += ar * br - ai * bi
                    ei += ar * bi + ai * br
                    d += abs(A[i, p]) * abs(B[p, j])
            assert abs(Fraction(C[i, j].real) - er) <= Fraction(d) * Fraction(1, 2 ** 52)
            assert abs(Fraction(C[i, j].imag) - ei) <= Fraction(d) * Fraction(1, 2 ** 52)
            assert abs(D[i, j] - d) <= 1e-15 * d
    # a transposed or swapped operand in the rank-2k wrappers would break Hermitian symmetry
    A, B = mk(6, 4), mk(6, 4)
    C2, D2 = direct.zher2k_dd(A, B)
    assert (np.abs(C2 - C2.conj().T) <= D2 * 2.0 ** -50).all()      # Hermitian up to the final rounding
    assert (np.abs(C2 - (A @ B.conj().T + B @ A.conj().T)) <= D2 * 1e-14).all()


@pytest.mark.parametrize("k", [6, 7, 1])
def test_syrk_is_real_part_of_herk_of_half_k(k):
    # Section 5: with Z = A1 + i A2, Z Z^H = A A^T + i (A2 A1^T - A1 A2^T); exact on integer data
    rng = np.random.default_rng(k)
    A = rng.integers(-9, 10, size=(5, k)).astype(np.float64)
    Bm = rng.integers(-9, 10, size=(5, k)).astype(np.float64)
    Z, ZB = staged.syrk_complexify(A), staged.syrk_complexify(Bm)
    assert Z.shape == (5, (k + 1) // 2)
    assert ((Z @ Z.conj().T).real == A @ A.T).all()
    assert ((Z @ ZB.conj().T + ZB @ Z.conj().T).real == A @ Bm.T + Bm @ A.T).all()          # SYR2K -> HER2K
    C, D = direct.dsyrk_dd(A)
    assert (C == A @ A.T).all()
    C2, _ = direct.dsyr2k_dd(A, Bm)
    assert (C2 == A @ Bm.T + Bm @ A.T).all()


def test_her2k_staged_symmetry_exactness_and_error():
    A = inputs.herk_input(9, 30, seed=15, dist="phi", phi=1.0)
    B = inputs.herk_input(9, 30, seed=16, dist="phi", phi=1.0)
    st = staged.zher2k2m_staged(A, B, 16)
    for Cp, Cm in st["Cpm"]:
        assert (Cm == Cp.T).all()                                    # Section 5: C- = C+^T
    assert (st["Xr"] == st["Xr"].T).all() and (st["Xi"] == -st["Xi"].T).all()
    assert all(abs(int(v)) <= 2 ** st["Pt"] for v in st["Xr"].ravel()) and all(abs(int(v)) <= 2 ** st["Pt"] for v in st["Xi"].ravel())
    # the 2M route reproduces the plain integer rank-2k update of the quantised matrices
    Ar, Ai = (q.astype(object) for q in st["Aq"])
    Br, Bi = (q.astype(object) for q in st["Bq"])
    Xr = Ar @ Br.T + Ai @ Bi.T + Br @ Ar.T + Bi @ Ai.T
    Xi = Ai @ Br.T - Ar @ Bi.T + Bi @ Ar.T - Br @ Ai.T
    assert (st["Xr"] == Xr).all() and (st["Xi"] == Xi).all()
    Cref, D = direct.zher2k_dd(A, B)
    assert direct.componentwise_error(st["C"], Cref, D) <= 1e-14


# ------------------------------------------------------------------ hybrid 2M/3M (Section 3 remark, Section 4)
def test_hybrid_moduli_extend_the_2m_set_with_coprime_non_2m_moduli(printed):
    h = staged.hybrid_moduli(26)
    assert h[:22] == staged.greedy_2m_moduli()
    assert h[22:] == [256, 253, 251, 249]
    assert all(not staged.is_2m_modulus(q) for q in h[22:])
    assert all(math.gcd(a, b) == 1 for i, a in enumerate(h) for b in h[:i])
    # greedy: every number between two consecutive extras shares a factor with something kept before it
    for hi, lo in zip([257] + h[22:-1], h[22:]):
        for cand in range(lo + 1, hi):
            kept_before = h[:h.index(lo)]
            assert any(math.gcd(cand, q) != 1 for q in kept_before), cand
    # 256, 253 and 251 are printed in the paper's real-modulus list; 255 and 247 clash with the 2M moduli 205/221
    real = set(printed["mreal_prefix"])
    assert {256, 253, 251} <= real and math.gcd(255, 205) == 5 and math.gcd(247, 221) == 13
    assert staged.hybrid_moduli(16) == staged.greedy_2m_moduli()[:16]
    assert staged.roots_of(h)[:22] == [staged.sqrt_minus_one(q) for q in h[:22]] and staged.roots_of(h)[22:] == [None] * 4


def test_symmetric_range_for_even_modulus_and_even_product():
    x = np.arange(-1000, 1000)
    r = staged.sym(x, 256)
    assert r.min() == -128 and r.max() == 127 and ((r - x) % 256 == 0).all()
    assert staged.sym(128, 256) == -128 and staged.sym(127, 256) == 127 and staged.sym(-128, 256) == -128
    M = 256 * 253
    for X in (0, 1, M // 2 - 1, M // 2, M - 1, -M // 2):
        L = staged.lift(X % M, M)
        assert -M // 2 <= L < M // 2 and (L - X) % M == 0        # Algorithm 1 step 6: [-M/2, M/2)
    assert staged.lift(M // 2, M) == -M // 2


def test_3m_identity_brute_force():
    # Eq. (1) after the reduction modulo m equals the complex product mod m, for every small Gaussian integer pair
    # and for entries across the whole residue range
    for m in staged.hybrid_moduli(26)[22:]:
        vals = list(range(-3, 4)) + [m // 2 - 1, -(m // 2), 77, -101]
        for ar in vals:
            for ai in vals:
                a3 = staged.pre_3m(ar, ai, m)
                assert (a3[0] - ar) % m == 0 and (a3[1] - ai) % m == 0 and (a3[2] - ar - ai) % m == 0
                assert all(-(m // 2) <= v <= (m - 1) // 2 for v in a3)
                for br in (-2, 0, 1, 5, m // 2 - 1):
                    for bi in (-7, 0, 3, -(m // 2)):
                        b3 = staged.pre_3m(br, bi, m)
                        P = [staged.sym(x * y, m) for x, y in zip(a3, b3)]
                        cr, ci = staged.post_3m(P[0], P[1], P[2], m)
                        assert (cr - (ar * br - ai * bi)) % m == 0
                        assert (ci - (ar * bi + ai * br)) % m == 0
                        assert -(m // 2) <= cr <= (m - 1) // 2 and -(m // 2) <= ci <= (m - 1) // 2


def test_3m_hand_example():
    # m = 253 (no square root of -1: 253 = 11 * 23), a = 3 + 2i, b = 1 - 4i, ab = 11 - 10i:
    # P1 = 3, P2 = -8, P3 = (3 + 2)(1 - 4) = -15; real = P1 - P2 = 11, imaginary = P3 - P1 - P2 = -10
    a3, b3 = staged.pre_3m(3, 2, 253), staged.pre_3m(1, -4, 253)
    assert a3 == (3, 2, 5) and b3 == (1, -4, -3)
    P = [staged.sym(x * y, 253) for x, y in zip(a3, b3)]
    assert P == [3, -8, -15] and staged.post_3m(*P, 253) == (11, -10)
    with pytest.raises(ValueError):
        staged.sqrt_minus_one(253)


@pytest.mark.parametrize("nmod", [23, 24, 26])
def test_hybrid_integer_path_equals_exact_product(nmod):
    # entries large enough that the result needs the moduli beyond the 22nd: |c| < 2 k 2^(2 b) must stay below M/2
    rng = np.random.default_rng(nmod)
    m, n, k, bits = 6, 5, 9, 75
    big = lambda shape: np.array([int(rng.integers(-2 ** 62, 2 ** 62)) * 2 ** (bits - 62) + int(rng.integers(0, 2 ** 13))
                                  for _ in range(int(np.prod(shape)))], dtype=object).reshape(shape)
    Ar, Ai, Br, Bi = big((m, k)), big((m, k)), big((k, n)), big((k, n))
    st = staged.gemm2m_int_staged(Ar, Ai, Br, Bi, nmod)
    cr = Ar.dot(Br) - Ai.dot(Bi)          # exact: Python integers
    ci = Ar.dot(Bi) + Ai.dot(Br)
    assert max(abs(int(v)) for v in np.concatenate([cr.ravel(), ci.ravel()])) > staged.product(staged.greedy_2m_moduli()) // 2
    assert (st["Xr"] == cr).all() and (st["Xi"] == ci).all()
    assert len(st["Cpm"][22]) == 3 and len(st["Cpm"][0]) == 2
    # a wrong sign in the 3M post-processing, or 3M residues fed to the 2M formulas, cannot survive this: the last
    # modulus alone decides the top bits of the result


@pytest.mark.parametrize("nmod", [23, 26])
def test_hybrid_float_path_bound_and_error(nmod):
    A, B = inputs.complex_inputs(10, 7, 60, seed=3 + nmod, dist="phi", phi=4.0)     # wide exponent span
    st = staged.zgemm2m_staged(A, B, nmod)
    assert st["moduli"][22:] == [256, 253, 251, 249][: nmod - 22]
    assert st["PA"] + st["PB"] == st["Pt"] and 2 ** st["Pt"] <= (st["M"] - 1) // 2 < 2 ** (st["Pt"] + 1)
    assert all(abs(int(v)) <= 2 ** st["Pt"] for v in np.concatenate([st["Xr"].ravel(), st["Xi"].ravel()]))
    pairs = np.array([(i, j) for i in range(10) for j in range(7)])
    Xs, vals = staged.staged_samples(st, pairs)       # plain integer product of the quantised matrices
    assert all(int(st["Xr"][i, j]) == xr and int(st["Xi"][i, j]) == xi for (i, j), (xr, xi) in zip(pairs.tolist(), Xs))
    Cref, D = direct.zgemm4m_dd(A, B)
    assert direct.componentwise_error(st["C"], Cref, D) <= 2.0 ** -52
    # more moduli than 22 must not be worse than 22
    e22 = direct.componentwise_error(staged.zgemm2m_staged(A, B, 22)["C"], Cref, D)
    assert direct.componentwise_error(st["C"], Cref, D) <= e22


# ------------------------------------------------------------------ extended interface (alpha, beta, op)
def test_extended_definition_vs_exact_rationals_and_special_cases():
    rng = np.random.default_rng(5)
    m, n, k = 4, 3, 5
    C0 = rng.standard_normal((m, n)) + 1j * rng.standard_normal((m, n))
    alpha, beta = 0.75 - 1.5j, -0.5 + 0.25j
    F = Fraction
    cf = lambda z: (F(float(np.real(z))), F(float(np.imag(z))))
    for ta, tb in (("N", "N"), ("T", "N"), ("N", "C"), ("C", "T"), ("C", "C")):
        A = rng.standard_normal((m, k) if ta == "N" else (k, m)) + 1j * rng.standard_normal((m, k) if ta == "N" else (k, m))
        B = rng.standard_normal((k, n) if tb == "N" else (n, k)) + 1j * rng.standard_normal((k, n) if tb == "N" else (n, k))
        got, D = direct.zgemm_ex_dd(ta, tb, alpha, A, B, beta, C0)
        for i in range(m):
            for j in range(n):
                sr = si = F(0)
                for p in range(k):          # the definition, entry by entry, with op() spelled out by index
                    a = A[i, p] if ta == "N" else (A[p, i] if ta == "T" else np.conj(A[p, i]))
                    b_ = B[p, j] if tb == "N" else (B[j, p] if tb == "T" else np.conj(B[j, p]))
                    (ar, ai), (br, bi) = cf(a), cf(b_)
                    sr += ar * br - ai * bi
                    si += ar * bi + ai * br
                (alr, ali), (ber, bei), (cr, ci) = cf(alpha), cf(beta), cf(C0[i, j])
                er = alr * sr - ali * si + ber * cr - bei * ci
                ei = alr * si + ali * sr + ber * ci + bei * cr
                assert abs(F(float(got[i, j].real)) - er) <= F(float(D[i, j])) * F(1, 2 ** 50)
                assert abs(F(float(got[i, j].imag)) - ei) <= F(float(D[i, j])) * F(1, 2 ** 50)
    A = rng.standard_normal((m, k)) + 0j
    B = rng.standard_normal((k, n)) + 0j
    nanC = np.full((m, n), np.nan + 0j)
    P, _ = direct.zgemm4m_dd(A, B)
    assert (direct.zgemm_ex_dd("N", "N", 1, A, B, 0, nanC)[0] == P).all()              # beta = 0: C0 not referenced
    assert (direct.zgemm_ex_dd("N", "N", 0, A * np.nan, B, 2, C0)[0] == 2 * C0).all()   # alpha = 0: A, B not referenced
    assert (direct.zgemm_ex_dd("T", "T", 1, A.T.copy(), B.T.copy(), 0, None)[0] == P).all()        # stored transposed


# ------------------------------------------------------------------ 2-norm scaling rule
def test_2norm_scaling_keeps_the_overflow_bound_and_is_never_looser():
    A, B = inputs.complex_inputs(19, 11, 700, seed=12, dist="phi", phi=1.5)
    A[4, :] = 0
    A[7, :] = 0
    A[7, 13] = 3.0 - 4.0j                       # a single entry: the 2-norm is 5, the max-based rule budgets sqrt(2k) 4
    for nmod in (7, 16, 22, 25):
        st_max = staged.zgemm2m_staged(A, B, nmod, upto="pre")
        st = staged.zgemm2m_staged(A, B, nmod, upto="pre", scaling="2norm")
        assert st["eA"][4] == 0
        assert (st["eA"] <= st_max["eA"]).all() and (st["eB"] <= st_max["eB"]).all()
        assert (st_max["eA"] - st["eA"]).max() <= st["ck"] + 1
        assert st_max["eA"][7] - st["eA"][7] >= st["ck"] - 2          # nearly the whole sqrt(2k) factor comes back
        for (qr, qi), axis, P in ((st["Aq"], 1, st["PA"]), (st["Bq"], 0, st["PB"])):
            sq = (qr.astype(object) ** 2 + qi.astype(object) ** 2).sum(axis=axis)
            assert all(int(v) <= 4 ** P for v in sq)                  # what Cauchy-Schwarz needs
            # and tight: one more bit would break the bound for at least one row (the rule wastes < 2 bits: ceil to a
            # power of 4 and the 2^-20 rounding up)
            assert any(16 * int(v) > 4 ** P for v in sq if v)


def test_2norm_scaling_gains_accuracy_and_equals_the_integer_product():
    A, B = inputs.complex_inputs(12, 9, 2048, seed=9, dist="phi", phi=0.5)
    Cref, D = direct.zgemm4m_dd(A, B)
    err = {}
    for scaling in ("max", "2norm"):
        st = staged.zgemm2m_staged(A, B, 14, scaling=scaling)
        assert all(abs(int(v)) <= 2 ** st["Pt"] for v in np.concatenate([st["Xr"].ravel(), st["Xi"].ravel()]))
        pairs = np.array([(i, j) for i in range(12) for j in range(9)])
        Xs, _ = staged.staged_samples(st, pairs)                      # no wrap-around: equals the plain integer product
        assert all(int(st["Xr"][i, j]) == xr and int(st["Xi"][i, j]) == xi for (i, j), (xr, xi) in zip(pairs.tolist(), Xs))
        err[scaling] = direct.componentwise_error(st["C"], Cref, D)
    assert err["2norm"] * 4 <= err["max"]          # k = 2048: c_k = 6; about three bits per operand come back, and the error is
    # proportional to 2^e of each operand (truncation of one factor times the other factor), not to their product


# ------------------------------------------------------------------ real Ozaki-II scheme (Section 3.1)
def test_real_scheme_moduli_and_integer_exactness(printed):
    mods = staged.greedy_real_moduli()
    assert mods[:10] == printed["mreal_prefix"]
    assert all(math.gcd(a, c) == 1 for i, a in enumerate(mods) for c in mods[:i])
    rng = np.random.default_rng(8)
    # integer-valued inputs whose product fits M/2: the scheme must return the exact product (every step is exact)
    A = rng.integers(-1000, 1000, size=(7, 33)).astype(np.float64)
    B = rng.integers(-1000, 1000, size=(33, 5)).astype(np.float64)
    st = staged.dgemm_o2_staged(A, B, 15)
    assert (st["C"] == A @ B).all()
    assert all(abs(int(v)) <= 2 ** st["Pt"] for v in st["X"].ravel())
    exact = st["Aq"].astype(object).dot(st["Bq"].astype(object))             # no wrap-around: plain integer product
    assert (st["X"] == exact).all()
    sq = (st["Aq"].astype(object) ** 2).sum(axis=1)
    assert all(int(v) <= 4 ** st["PA"] for v in sq)                           # the row 2-norm bound of the scaling rule


def test_real_scheme_error_vs_modulus_count():
    rng = np.random.default_rng(9)
    A = (rng.random((10, 300)) - 0.5) * np.exp(0.5 * rng.standard_normal((10, 300)))
    B = (rng.random((300, 8)) - 0.5) * np.exp(0.5 * rng.standard_normal((300, 8)))
    Cref, D = direct.dgemm_dd(A, B)
    errs = [direct.componentwise_error(staged.dgemm_o2_staged(A, B, n)["C"], Cref, D) for n in (8, 12, 15)]
    assert errs[0] > 100 * errs[1] > 100 * errs[2] and errs[2] <= 1e-14      # 15 real moduli ~ 16 2M moduli (Section 4)
    # against exact rationals on a tiny case
    F = Fraction
    got, _ = direct.dgemm_dd(A[:3, :20], B[:20, :2])
    for i in range(3):
        for j in range(2):
            ex = sum(F(float(A[i, p])) * F(float(B[p, j])) for p in range(20))
            assert abs(F(float(got[i, j])) - ex) <= abs(ex) * F(1, 2 ** 52)

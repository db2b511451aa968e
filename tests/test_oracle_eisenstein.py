"""Pins of the Eisenstein-integer oracle (Sections 3.2 and 4) against what the mathematics fixes: the ring's multiplication
against complex arithmetic, the homomorphisms against that multiplication, the CRT path against a brute-force product over
Z[w], the fixed-point lattice rounding against the exact nearest-point definition and the lattice's packing and covering
radii, and the whole path against an independent double-double ZGEMM."""
from __future__ import annotations

import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import direct, eisenstein as E, staged

W = complex(-0.5, math.sqrt(3.0) / 2)


def test_moduli_are_the_primes_one_mod_three():
    mods = E.greedy_eisenstein_moduli()
    assert len(mods) == 23 and mods[0] == 247 and all(m < 256 for m in mods)
    for i, m in enumerate(mods):
        assert all(p % 3 == 1 for p in staged.prime_factors(m))
        assert all(math.gcd(m, q) == 1 for q in mods[:i])
    # the greedy set is maximal: every prime congruent to 1 mod 3 below 256 divides exactly one modulus, and no square does
    primes = [p for p in range(2, 256) if len(staged.prime_factors(p)) == 1 and p % 3 == 1]
    assert len(primes) == 25
    assert staged.product(mods) == math.prod(primes)
    # Section 4's qualitative statement: more bits than the Gaussian 2M set offers (2^152)
    bits_e = math.log2(staged.product(mods))
    bits_g = math.log2(staged.product(staged.greedy_2m_moduli()))
    assert bits_e > bits_g and abs(bits_g - 152.08) < 0.01 and abs(bits_e - 160.88) < 0.01


def test_excluded_moduli_have_no_usable_root_pair():
    for m in (3, 9, 21, 5, 11, 25, 255, 256):       # 3 ramifies (double root), 21 = 3 * 7, the rest have an inert prime
        roots = [s for s in range(m) if (s * s + s + 1) % m == 0]
        usable = [s for s in roots if math.gcd((s - s * s) % m, m) == 1]
        assert not usable and not E.is_eisenstein_modulus(m)


def test_cube_roots():
    for m in E.greedy_eisenstein_moduli():
        s = E.cube_root_of_unity(m)
        assert (s * s + s + 1) % m == 0 and pow(s, 3, m) == 1 and s != 1
        assert ((s - s * s) ** 2 + 3) % m == 0                  # s - s^2 is a square root of -3
        assert all((r * r + r + 1) % m for r in range(2, s))    # the smallest one


def test_ring_multiplication_is_complex_multiplication():
    rng = np.random.default_rng(1)
    for _ in range(200):
        a, b, c, d = (int(v) for v in rng.integers(-1000, 1000, 4))
        pa, pb = E.eis_mul(a, b, c, d)
        assert abs((a + b * W) * (c + d * W) - (pa + pb * W)) < 1e-6
    assert E.eis_mul(0, 1, 0, 1) == (-1, -1)                    # w^2 = -1 - w
    assert E.eis_mul(1, 1, 1, 1) == (0, 1)                      # (1 + w)^2 = (-w^2)^2 = w


def test_homomorphisms_and_inverse():
    rng = np.random.default_rng(2)
    for m in (247, 217, 37):
        s = E.cube_root_of_unity(m)
        a, b, c, d = (rng.integers(-10**6, 10**6, 50) for _ in range(4))
        xp, xm = E.pre_e(a % m, b % m, m, s)
        yp, ym = E.pre_e(c % m, d % m, m, s)
        pa, pb = E.eis_mul(a, b, c, d)
        zp, zm = E.pre_e(pa % m, pb % m, m, s)
        assert np.all((xp * yp - zp) % m == 0) and np.all((xm * ym - zm) % m == 0)
        ra, rb = E.post_e(zp, zm, m, s)
        assert np.all((ra - pa) % m == 0) and np.all((rb - pb) % m == 0)
        assert np.all(np.abs(ra) <= (m - 1) // 2) and np.all(np.abs(xp) <= (m - 1) // 2)


@pytest.mark.parametrize("nmod,bits", [(2, 5), (5, 15), (12, 40), (23, 70)])
def test_crt_path_equals_brute_force_product(nmod, bits):
    rng = np.random.default_rng(nmod)
    m, k, n = 4, 6, 3
    draw = lambda shape: np.array([[int(rng.integers(-2**31, 2**31)) * (1 << max(bits - 31, 0)) >> max(31 - bits, 0)
                                    for _ in range(shape[1])] for _ in range(shape[0])], dtype=object)
    Aa, Ab, Ba, Bb = draw((m, k)), draw((m, k)), draw((k, n)), draw((k, n))
    st = E.eisenstein_int_staged(Aa, Ab, Ba, Bb, nmod)
    Ca, Cb = E.eis_matmul(Aa, Ab, Ba, Bb)
    bound = max(abs(int(v)) for v in np.concatenate([Ca.ravel(), Cb.ravel()]))
    assert 2 * bound < st["M"], "test sized inside the budget"
    assert np.all(st["Xa"] == Ca) and np.all(st["Xb"] == Cb)


def test_crt_path_wraps_modulo_M_outside_the_budget():
    rng = np.random.default_rng(7)
    Aa, Ab = (rng.integers(-2**20, 2**20, (3, 4)).astype(object) for _ in range(2))
    Ba, Bb = (rng.integers(-2**20, 2**20, (4, 3)).astype(object) for _ in range(2))
    st = E.eisenstein_int_staged(Aa, Ab, Ba, Bb, 2)              # M = 247 * 241 is far too small
    Ca, Cb = E.eis_matmul(Aa, Ab, Ba, Bb)
    assert np.any(st["Xa"] != Ca)
    assert all((int(x) - int(c)) % st["M"] == 0 for x, c in zip(st["Xa"].ravel(), Ca.ravel()))


def test_lattice_points_within_the_packing_radius_round_to_themselves():
    # the hexagonal lattice has packing radius 1/2: any z with |z - p| < 1/2 has p as its unique nearest point
    rng = np.random.default_rng(3)
    for mag in (3, 1000, 2**40):
        for _ in range(300):
            a, b = int(rng.integers(-mag, mag)), int(rng.integers(-mag, mag))
            r, th = 0.49 * rng.random(), 2 * math.pi * rng.random()
            # as doubles: at 2^40 the roundings of x and y move the point by 2^-12 at most, still inside the radius
            x = (a - b / 2 + r * math.cos(th))
            y = (b * math.sqrt(3.0) / 2 + r * math.sin(th))
            assert E.quantise_hex_one(x, y, 0) == (a, b)
            assert E.nearest_eisenstein_exact(Fraction(x), Fraction(y)) == (a, b)
    assert E.quantise_hex_one(0.0, 0.0, 0) == (0, 0)
    assert E.quantise_hex_one(-0.5, math.sqrt(3.0) / 2, 0) == (0, 1)            # w itself
    assert E.quantise_hex_one(0.5, 3 * math.sqrt(3.0) / 2, 0) == (2, 3)         # 2 + 3w
    assert E.quantise_hex_one(-2.0, -4 * math.sqrt(3.0), -1) == (-12, -16)       # 2 (-2 - 4 sqrt(3) i) = -12 - 16w


def test_fixed_point_rounding_against_the_exact_definition():
    rng = np.random.default_rng(4)
    rho = 1 / math.sqrt(3.0)
    worst, differ = 0.0, 0
    for trial in range(1500):
        e = int(rng.integers(-30, 30))
        big = trial % 3 == 0
        x = float(rng.standard_normal()) * (2.0 ** (60 if big else 4))
        y = float(rng.standard_normal()) * (2.0 ** (60 if big else 4))
        X, Y = Fraction(x) / Fraction(2) ** e, Fraction(y) / Fraction(2) ** e
        got = E.quantise_hex_one(x, y, e)
        want = E.nearest_eisenstein_exact(X, Y)
        dg = E.distance_to(X, Y, *got)
        worst = max(worst, dg)
        if got != want:
            # only within the fixed-point resolution of a boundary; doubles above 2^53 have no fraction bits, so there the
            # two half-odd neighbours of an integer X tie exactly and either choice is a nearest point
            assert dg - E.distance_to(X, Y, *want) < 2.0 ** -25
            differ += 0 if big else 1
    assert differ <= 2
    assert worst <= rho + 2.0 ** -25 and worst > 0.9 * rho           # covering radius of the hexagonal lattice


def test_deep_holes_and_edges():
    # the deep hole (1/2, 1/(2 sqrt 3)) is equidistant from 0, 1 and 1 + w: any of them is valid, at distance 1/sqrt 3
    x, y = 0.5, 0.5 / math.sqrt(3.0)
    a, b = E.quantise_hex_one(x, y, 0)
    assert (a, b) in ((0, 0), (1, 0), (1, 1))
    assert abs(E.distance_to(Fraction(x), Fraction(y), a, b) - 1 / math.sqrt(3.0)) < 1e-9
    # reflections: the choice for (-x, y), (x, -y) mirrors the choice for (x, y)
    rng = np.random.default_rng(5)
    for _ in range(200):
        x, y = float(rng.standard_normal()) * 50, float(rng.standard_normal()) * 50
        a, b = E.quantise_hex_one(x, y, 0)
        u, v = 2 * a - b, b
        a2, b2 = E.quantise_hex_one(-x, y, 0)
        assert (2 * a2 - b2, b2) == (-u, v)
        a3, b3 = E.quantise_hex_one(x, -y, 0)
        assert (2 * a3 - b3, b3) == (u, -v)


def test_scaling_budget_holds_for_adversarial_inputs():
    # all parts at the row maximum with the signs that align every term: the product's coordinates must stay inside the lift
    for nmod, k in ((2, 4), (3, 64), (6, 1024), (23, 300)):
        mods = E.greedy_eisenstein_moduli()[:nmod]
        M = staged.product(mods)
        Pt, PA, PB, ck = E.scaling_targets_e(M, k)
        if PB - ck < 2:
            continue
        assert 4 ** ck >= 5 * k > 4 ** (ck - 1) and PA + PB == Pt and 2 ** Pt <= (M - 1) // 2 < 2 ** (Pt + 1)
        for ph in (1 + 1j, 1 - 1j, 1j, 1.0, 0.999 + 0.57j):
            A = np.full((2, k), ph * 1.9999, dtype=np.complex128)
            B = np.full((k, 2), np.conj(ph) * 1.9999, dtype=np.complex128)
            st = E.zgemm_eisenstein_staged(A, B, nmod, upto="pre")
            Ca, Cb = E.eis_matmul(st["Aq"][0], st["Aq"][1], st["Bq"][0], st["Bq"][1]) if k <= 64 else (None, None)
            if Ca is not None:
                assert np.all(st["Xa"] == Ca) and np.all(st["Xb"] == Cb)
            for X in (st["Xa"], st["Xb"], 2 * st["Xa"] - st["Xb"]):
                assert max(abs(int(v)) for v in X.ravel()) <= 2 ** Pt or Ca is None


def test_real_integer_inputs_are_multiplied_exactly():
    rng = np.random.default_rng(6)
    A = rng.integers(-1000, 1000, (5, 12)).astype(np.float64) * (2.0 ** rng.integers(-8, 8, (5, 1)))
    B = rng.integers(-1000, 1000, (12, 4)).astype(np.float64)
    st = E.zgemm_eisenstein_staged(A.astype(np.complex128), B.astype(np.complex128), 8)
    assert np.all(st["C"].imag == 0) and np.all(st["C"].real == A @ B)     # real integers lie on the lattice (b = 0)


def test_conversion_of_the_result():
    Ca = np.array([[3, -7, 2**80 + 12345]], dtype=object)
    Cb = np.array([[4, 5, -(2**79) + 999]], dtype=object)
    out = E.unscale_e(Ca, Cb, [1], [2, 2, 2])
    for j in range(3):
        a, b = int(Ca[0, j]), int(Cb[0, j])
        re = Fraction(2 * a - b, 2) * 8
        assert abs(Fraction(out[0, j].real) - re) <= abs(re) * Fraction(1, 2**53)
        # Im^2 = 3 b^2 / 4 * 64 exactly; the rounded value squared must agree to the precision of one rounding
        im2 = Fraction(3 * b * b, 4) * 64
        assert abs(Fraction(out[0, j].imag) ** 2 - im2) <= im2 * Fraction(3, 2**53)
        assert (out[0, j].imag > 0) == (b > 0)


@pytest.mark.parametrize("nmod,tol", [(8, 2.0 ** -24), (12, 2.0 ** -38), (16, 2.0 ** -50), (23, 2.0 ** -50)])
def test_whole_path_against_double_double(nmod, tol):
    rng = np.random.default_rng(nmod)
    A = rng.standard_normal((9, 40)) + 1j * rng.standard_normal((9, 40))
    B = rng.standard_normal((40, 7)) + 1j * rng.standard_normal((40, 7))
    A *= 2.0 ** rng.integers(-20, 20, (9, 1))
    st = E.zgemm_eisenstein_staged(A, B, nmod)
    ref, D = direct.zgemm4m_dd(A, B)
    assert np.max(np.abs(st["C"] - ref) / D) < tol
    if nmod == 8:                                    # ... and not better than the quantisation allows: the bound is not vacuous
        assert np.max(np.abs(st["C"] - ref) / D) > 2.0 ** -40

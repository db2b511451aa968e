"""The Eisenstein-integer analogue of Algorithm 1 (Sections 3.2 and 4) in exact integers -- TEST INFRASTRUCTURE ONLY.

Section 3.2 replaces the Gaussian integers Z[i] by the Eisenstein integers Z[w], w = exp(2 pi i / 3), w^2 + w + 1 = 0;
Section 4 adds that quantisation then rounds every point of the complex plane to the nearest point of the hexagonal
lattice.  Everything else is Algorithm 1 with the ring changed, written here in the ring's own basis {1, w}:

  is_eisenstein_modulus, greedy_eisenstein_moduli   the 2M condition for Z[w]: x^2 + x + 1 has two roots s, s^2 modulo m
                                    that differ by a unit, i.e. m is a product of primes congruent to 1 mod 3; greedy
                                    coprime walk down from 256 as in Section 4
  cube_root_of_unity                s with s^2 + s + 1 = 0 (mod m)
  eis_mul                           (a + b w)(c + d w) = (ac - bd) + (ad + bc - bd) w
  pre_e, post_e                     the analogues of Eq. (2a), (2c): the two ring homomorphisms w -> s and w -> s^2, and the
                                    inverse map
  nearest_eisenstein_exact          nearest lattice point by exact arithmetic (the definition)
  quantise_hex                      nearest lattice point by the fixed-point procedure below (what an implementation can
                                    reproduce bit for bit); pinned against the definition in the tests
  zgemm_eisenstein_staged           the whole path

Parity unpinned: `greedy_eisenstein_moduli` against the paper.  Section 4 prints one figure for this variant, M ~ 2^154.5
for the 8-bit moduli; the set defined here (every prime congruent to 1 mod 3 below 256 divides exactly one modulus) has
M = 2^160.9, and no reading of the walk tried reproduces the printed figure.  The set is pinned by its definition and the
qualitative claim (more bits than the Gaussian set's 2^152) only; everything else in this file is pinned by the tests.

Readings (the paper only sketches this variant):
  * s is the smallest positive root;
  * scale factors as in Algorithm 1 step 2 from the largest |Re|, |Im| of a row / column, with c_k = ceil(log2(5k)/2):
    the scaled parts stay below T = 2^(P - c_k) >= 4, a lattice point within rho = 0.578 of z has |z'| <= sqrt(2) T + rho
    <= 1.1021 sqrt(2) T, so |c| <= 2.43 k 2^(P_t - 2 c_k) for every entry c of the product and every coordinate of c in
    {1, w} or in {1, sqrt(-3)}/2 is at most 2|c| <= 2^P_t <= (M-1)/2;
  * quantisation: X = |Re z| 2^-e and t = |Im z| 2^-e (2/sqrt 3) are taken as fixed-point numbers with 32 fractional bits
    (floor), the factor 2/sqrt 3 as the 128-bit constant floor(2^127 2/sqrt 3).  The lattice is the union of the points
    (u + v sqrt(-3))/2 with u, v both even and with u, v both odd; the nearest point of the first kind has
    u0 = 2 rn(X), v0 = 2 rn(t/2), and it beats the nearest point of the second kind (u1 = 2 floor(X) + 1,
    v1 = 2 floor(t/2) + 1) exactly when |X - u0/2| + (3/2) |t - v0| <= 1 (the squared distance is dx^2 + (3/4) dt^2, and the
    second kind's deviations are 1/2 - |dx| and 1 - |dt|);
    the signs of Re z and Im z are then applied to u and v (the lattice is symmetric under both reflections).  In the
    basis {1, w}: b = v, a = (u + v)/2;
  * the result a + b w is converted with one rounding per part: Re = (2a - b)/2, Im = b sqrt(3)/2.
"""
from __future__ import annotations

import math
from fractions import Fraction

import numpy as np

from . import staged

FRAC_BITS = 32
K3_BITS = 127
K3 = math.isqrt((4 << (2 * K3_BITS)) // 3)         # floor(2^127 * 2 / sqrt(3)) = floor(sqrt(4/3 * 4^127))


# ----------------------------------------------------------------------------- moduli (Sections 3.2, 4)
def is_eisenstein_modulus(m: int) -> bool:
    """x^2 + x + 1 splits into two roots that differ by a unit modulo m: every prime factor is congruent to 1 mod 3."""
    return m > 1 and all(p % 3 == 1 for p in staged.prime_factors(m))


def greedy_eisenstein_moduli(limit: int = 256):
    kept = []
    for cand in range(limit, 1, -1):
        if is_eisenstein_modulus(cand) and all(math.gcd(cand, q) == 1 for q in kept):
            kept.append(cand)
    return kept


def cube_root_of_unity(m: int) -> int:
    for s in range(2, m):
        if (s * s + s + 1) % m == 0:
            return s
    raise ValueError(f"{m} is not an Eisenstein 2M modulus")


# ----------------------------------------------------------------------------- the ring
def eis_mul(a, b, c, d):
    """(a + b w)(c + d w) with w^2 = -1 - w."""
    return a * c - b * d, a * d + b * c - b * d


def eis_matmul(Aa, Ab, Ba, Bb):
    """Exact product of matrices over Z[w], entry by entry from `eis_mul` (object arrays of Python ints)."""
    m, k = Aa.shape
    n = Ba.shape[1]
    Ca = np.zeros((m, n), dtype=object)
    Cb = np.zeros((m, n), dtype=object)
    for i in range(m):
        for j in range(n):
            sa, sb = 0, 0
            for l in range(k):
                pa, pb = eis_mul(int(Aa[i, l]), int(Ab[i, l]), int(Ba[l, j]), int(Bb[l, j]))
                sa += pa
                sb += pb
            Ca[i, j], Cb[i, j] = sa, sb
    return Ca, Cb


def pre_e(Xa, Xb, m: int, s: int):
    """Analogue of Eq. (2a): the images of X = Xa + Xb w under w -> s and w -> s^2 (the conjugate root)."""
    s2 = (s * s) % m
    return staged.sym(Xa + s * Xb, m), staged.sym(Xa + s2 * Xb, m)


def post_e(Cp, Cm, m: int, s: int):
    """Analogue of Eq. (2c): from c_a + s c_b = C+ and c_a + s^2 c_b = C-:  c_b = (C+ - C-)/(s - s^2), c_a = C+ - s c_b."""
    s2 = (s * s) % m
    dinv = pow((s - s2) % m, -1, m)
    cb = ((Cp - Cm) * dinv) % m
    ca = (Cp - s * cb) % m
    return staged.sym(ca, m), staged.sym(cb, m)


# ----------------------------------------------------------------------------- quantisation (Section 4)
def _sign_p_plus_q_sqrt3(p: Fraction, q: Fraction) -> int:
    """Sign of p + q sqrt(3), exactly."""
    if p == 0 and q == 0:
        return 0
    if p >= 0 and q >= 0:
        return 1
    if p <= 0 and q <= 0:
        return -1
    big_p = p * p > 3 * q * q
    return (1 if p > 0 else -1) if big_p else (1 if q > 0 else -1)


def nearest_eisenstein_exact(X: Fraction, Y: Fraction):
    """The definition: (a, b) minimising |X + iY - (a + b w)|^2 = (X - a + b/2)^2 + (Y - b sqrt(3)/2)^2, decided exactly.
    |.|^2 = R(a, b) - sqrt(3) Y b with R rational, so two candidates compare through the sign of p + q sqrt(3)."""
    scale = 1 << 200
    b0 = int((2 * Y * scale) // math.isqrt(3 * scale * scale))          # about 2Y / sqrt(3)
    best = None
    for b in range(b0 - 2, b0 + 4):
        a0 = math.floor(X + Fraction(b, 2))
        for a in (a0 - 1, a0, a0 + 1, a0 + 2):
            R = (X - a + Fraction(b, 2)) ** 2 + Y * Y + Fraction(3 * b * b, 4)
            if best is None:
                best = (R, a, b)
                continue
            # d^2(cand) - d^2(best) = (R - R_best) - sqrt(3) Y (b - b_best)
            if _sign_p_plus_q_sqrt3(R - best[0], -Y * (b - best[2])) < 0:
                best = (R, a, b)
    return best[1], best[2]


def distance_to(X: Fraction, Y: Fraction, a: int, b: int) -> float:
    """|X + iY - (a + b w)| in floating point (for bounds, not for decisions)."""
    dx = float(X - a + Fraction(b, 2))
    dy = float(Y - Fraction(b * math.isqrt(3 << 400), 1 << 201))        # sqrt(3)/2 to 200 bits
    return math.hypot(dx, dy)


def _fixed_floor(v: float, e: int, extra: int = 1, extra_shift: int = 0) -> int:
    """floor(|v| 2^-e extra 2^(FRAC_BITS - extra_shift)) exactly."""
    fr = Fraction(abs(float(v)))
    num = fr.numerator * extra
    sh = FRAC_BITS - extra_shift - e
    if sh >= 0:
        return (num << sh) // fr.denominator
    return num // (fr.denominator << (-sh))


def quantise_hex_one(x: float, y: float, e: int):
    """(a, b) of the lattice point chosen for (x + iy) 2^-e by the fixed-point procedure of the module header."""
    one = 1 << FRAC_BITS
    Xf = _fixed_floor(x, e)
    Tf = _fixed_floor(y, e, K3, K3_BITS)
    n0 = (Xf + one // 2) >> FRAC_BITS                 # rn(X)
    h0 = (Tf + one) >> (FRAC_BITS + 1)                # rn(t/2)
    dx0 = abs(Xf - (n0 << FRAC_BITS))
    dt0 = abs(Tf - (h0 << (FRAC_BITS + 1)))
    if 2 * dx0 + 3 * dt0 <= 2 * one:
        u, v = 2 * n0, 2 * h0
    else:
        u, v = 2 * (Xf >> FRAC_BITS) + 1, 2 * (Tf >> (FRAC_BITS + 1)) + 1
    if x < 0:
        u = -u
    if y < 0:
        v = -v
    return (u + v) // 2, v


def quantise_hex(Z, e, axis: int):
    """Step 3 for the hexagonal lattice: (Za, Zb) with Z 2^-e ~ Za + Zb w; e per row (axis=1) or column (axis=0)."""
    Z = np.asarray(Z, dtype=np.complex128)
    Za = np.zeros(Z.shape, dtype=object)
    Zb = np.zeros(Z.shape, dtype=object)
    for i in range(Z.shape[0]):
        for j in range(Z.shape[1]):
            ee = int(e[i] if axis == 1 else e[j])
            Za[i, j], Zb[i, j] = quantise_hex_one(float(Z[i, j].real), float(Z[i, j].imag), ee)
    return Za, Zb


# ----------------------------------------------------------------------------- scaling and conversion (steps 2, 7)
def scaling_targets_e(M: int, k: int):
    """P_t = floor(log2((M-1)/2)) split as in Algorithm 1; c_k = ceil(log2(5k)/2) (see the module header)."""
    Pt = ((M - 1) // 2).bit_length() - 1
    PA, PB = (Pt + 1) // 2, Pt // 2
    ck = 0
    while 4 ** ck < 5 * max(k, 1):
        ck += 1
    return Pt, PA, PB, ck


_SQRT3_BITS = 300
_SQRT3 = math.isqrt(3 << (2 * _SQRT3_BITS))          # floor(sqrt(3) 2^300)


def unscale_e(Ca, Cb, e_row, f_col, bits: int = 53):
    """Step 7: (c_a + c_b w) sigma_i tau_j = ((2 c_a - c_b)/2 + i c_b sqrt(3)/2) 2^(e_i + f_j), one rounding per part."""
    m, n = Ca.shape
    out = np.zeros((m, n), dtype=np.complex128)
    for i in range(m):
        for j in range(n):
            ex = int(e_row[i]) + int(f_col[j])
            yr, tr = staged.round_int_nearest_even(2 * int(Ca[i, j]) - int(Cb[i, j]), bits)
            yi, ti = staged.round_int_nearest_even(int(Cb[i, j]) * _SQRT3, bits)
            out[i, j] = complex(math.ldexp(float(yr), tr + ex - 1), math.ldexp(float(yi), ti + ex - 1 - _SQRT3_BITS))
    return out


# ----------------------------------------------------------------------------- whole path
def _planes(Za, Zb, moduli, roots):
    Za, Zb = staged._small(Za), staged._small(Zb)
    out = []
    for ml, sl in zip(moduli, roots):
        p, q = pre_e(Za % ml, Zb % ml, ml, sl)
        out.append((np.asarray(p).astype(np.int64), np.asarray(q).astype(np.int64)))
    return out


def eisenstein_int_staged(Aa, Ab, Ba, Bb, nmod: int):
    """Integer matrices over Z[w] (coefficients of 1 and w): 2M multiplication with the ring homomorphisms w -> s, s^2 and
    CRT over the first `nmod` Eisenstein moduli.  Exact while every coefficient of the product is below M/2."""
    moduli = greedy_eisenstein_moduli()[:nmod]
    roots = [cube_root_of_unity(q) for q in moduli]
    M = staged.product(moduli)
    Apl = _planes(np.asarray(Aa).astype(object), np.asarray(Ab).astype(object), moduli, roots)
    Bpl = _planes(np.asarray(Ba).astype(object), np.asarray(Bb).astype(object), moduli, roots)
    Cpm, res_a, res_b = [], [], []
    for Ap, Bp, ml, sl in zip(Apl, Bpl, moduli, roots):
        Cp, Cm = staged.mul_2m(Ap[0], Bp[0], ml), staged.mul_2m(Ap[1], Bp[1], ml)
        Cpm.append((Cp, Cm))
        ca, cb = post_e(Cp, Cm, ml, sl)
        res_a.append(ca)
        res_b.append(cb)
    Xa, Xb = staged.lift(staged.crt(res_a, moduli), M), staged.lift(staged.crt(res_b, moduli), M)
    return dict(moduli=moduli, roots=roots, M=M, Apm=Apl, Bpm=Bpl, Cpm=Cpm, Xa=Xa, Xb=Xb)


def zgemm_eisenstein_staged(A, B, nmod: int, out_bits: int = 53, upto: str = "all"):
    """The Eisenstein analogue of Algorithm 1 on floating-point A (m x k), B (k x n)."""
    A = np.asarray(A)
    B = np.asarray(B)
    k = A.shape[1]
    moduli = greedy_eisenstein_moduli()[:nmod]
    M = staged.product(moduli)
    Pt, PA, PB, ck = scaling_targets_e(M, k)
    if PB - ck < 2:
        raise ValueError("too few moduli for this k")
    eA = staged.scaling_exponents(A, 1, PA, ck)
    eB = staged.scaling_exponents(B, 0, PB, ck)
    Aq = quantise_hex(A, eA, 1)
    Bq = quantise_hex(B, eB, 0)
    st = dict(moduli=moduli, M=M, Pt=Pt, PA=PA, PB=PB, ck=ck, eA=eA, eB=eB, Aq=Aq, Bq=Bq)
    if upto == "quantise":
        return st
    st.update(eisenstein_int_staged(Aq[0], Aq[1], Bq[0], Bq[1], nmod))
    if upto == "pre":
        return st
    st["C"] = unscale_e(st["Xa"], st["Xb"], eA, eB, out_bits)
    return st

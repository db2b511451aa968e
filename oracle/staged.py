"""Algorithm 1 ("2M Ozaki-II") step by step in exact integers -- TEST INFRASTRUCTURE ONLY.

Every function follows one passage of the paper, in its notation, with no blocking or fusion:

  is_2m_modulus, greedy_2m_moduli   Section 2 (definition of a 2M modulus) and Section 4 (greedy coprime set in [1, 256])
  sqrt_minus_one, inv2              Section 2: s^2 = -1 (mod m); 2^-1 = (m+1)/2
  pre_2m, mul_2m, post_2m           Eq. (2a), (2b), (2c)
  greedy_real_moduli, dgemm_o2_staged      Section 3.1 (the real Ozaki-II scheme) with the real modulus set of Section 4
  hybrid_moduli, pre_3m, mul_3m, post_3m   Section 3 (hybrid 2M/3M remark) and Section 4 (non-2M moduli once the 2M set is
                                    exhausted); Eq. (1) applied after the reduction modulo m
  crt, lift                         Section 3.1 (CRT formula) and Algorithm 1 steps 5-6
  scaling_targets, scaling_exponents, quantise, unscale   Algorithm 1 steps 2, 3, 7

Readings taken where the paper is silent (they are the library's documented readings too):
  * s is the smallest positive root (any root gives the same C);
  * residues are kept as symmetric representatives in [-(m-1)/2, (m-1)/2] (even m, hybrid only: [-m/2, m/2 - 1]);
  * hybrid: all 22 2M moduli first, then the greedy walk down from 256 over the remaining coprime (non-2M) moduli;
  * scale factors are powers of two chosen from the largest part-magnitude of each row of A /
    column of B so that every entry of the integer product is bounded by 2^P_t <= (M-1)/2
    (Cauchy-Schwarz), see `scaling_exponents`;
  * quantisation truncates toward zero (keeps that bound rigorous);
  * the CRT sum is reduced mod M and lifted to [-(M-1)/2, (M-1)/2];
  * the lifted integer is rounded once (nearest-even) to the output precision, then scaled by 2^(e_i+f_j).
"""
from __future__ import annotations

import math

import numpy as np


# ----------------------------------------------------------------------------- moduli (Sections 2, 4)
def prime_factors(n: int):
    out = []
    p = 2
    while p * p <= n:
        while n % p == 0:
            out.append(p)
            n //= p
        p += 1
    if n > 1:
        out.append(n)
    return out


def is_2m_modulus(m: int) -> bool:
    """Section 2: m odd and a product of primes congruent to 1 mod 4 (equivalently s with s^2 = -1 exists)."""
    return m > 1 and m % 2 == 1 and all(p % 4 == 1 for p in prime_factors(m))


def greedy_2m_moduli(limit: int = 256):
    """Section 4: walk down from `limit`, keep every 2M modulus coprime to all those already kept."""
    kept = []
    for cand in range(limit, 1, -1):
        if is_2m_modulus(cand) and all(math.gcd(cand, q) == 1 for q in kept):
            kept.append(cand)
    return kept


def greedy_real_moduli(limit: int = 256):
    """Section 4, the set available to real Ozaki-II GEMMs: the same greedy walk without the 2M condition."""
    kept = []
    for cand in range(limit, 1, -1):
        if all(math.gcd(cand, q) == 1 for q in kept):
            kept.append(cand)
    return kept


def sqrt_minus_one(m: int) -> int:
    """Smallest positive s with s^2 = -1 (mod m) (Section 2)."""
    for s in range(1, m):
        if (s * s + 1) % m == 0:
            return s
    raise ValueError(f"{m} is not a 2M modulus")


def inv2(m: int) -> int:
    """Section 2: 2^-1 = (m+1)/2 mod m."""
    return (m + 1) // 2


def sym(x, m: int):
    """Symmetric representative of x mod m: in [-(m-1)/2, (m-1)/2] for odd m, in [-m/2, m/2 - 1] for even m."""
    h = m // 2
    return (x + h) % m - h


def hybrid_moduli(n: int, limit: int = 256):
    """Sections 3 and 4: the 2M moduli first; when they are exhausted, further moduli come from the same greedy walk
    down from `limit` over the numbers coprime to everything kept (none of them is a 2M modulus, or the first walk
    would have kept it).  Returns the first n moduli."""
    kept = greedy_2m_moduli(limit)
    if n > len(kept):
        for cand in range(limit, 1, -1):
            if len(kept) >= n:
                break
            if all(math.gcd(cand, q) == 1 for q in kept):
                kept.append(cand)
    return kept[:n]


# ----------------------------------------------------------------------------- 2M multiplication (Eq. 2a-2c)
def pre_2m(Xr, Xi, m: int, s: int):
    """Eq. (2a): X+ = Xr + s Xi, X- = Xr - s Xi (mod m), symmetric representatives."""
    return sym(Xr + s * Xi, m), sym(Xr - s * Xi, m)


def _exact_matmul(P, Q):
    """Exact integer matrix product of small-integer matrices (a library matmul used as one step)."""
    P = np.asarray(P)
    Q = np.asarray(Q)
    k = P.shape[1]
    pm = int(np.abs(P).max(initial=0))
    qm = int(np.abs(Q).max(initial=0))
    if max(k, 1) * pm * qm < 2 ** 52:              # exact in float64, BLAS does the work
        return np.rint(P.astype(np.float64) @ Q.astype(np.float64)).astype(np.int64)
    return P.astype(object) @ Q.astype(object)


def mul_2m(Ap, Bp, m: int):
    """Eq. (2b): C+- = A+- B+- (mod m)."""
    return sym(_exact_matmul(Ap, Bp), m)


def post_2m(Cp, Cm, m: int, s: int):
    """Eq. (2c): C = 2^-1 (C- + C+) + i s 2^-1 (C- - C+) (mod m)."""
    h = inv2(m)
    return sym(h * (Cm + Cp), m), sym(s * h * (Cm - Cp), m)


# ----------------------------------------------------------------------------- 3M multiplication modulo m (Eq. 1, Section 3)
def pre_3m(Xr, Xi, m: int):
    """Residues of Xr, Xi and Xr + Xi (the sum is formed after the reduction, Section 3)."""
    r, i = sym(Xr, m), sym(Xi, m)
    return r, i, sym(r + i, m)


def mul_3m(A3, B3, m: int):
    """The three real products of Eq. (1) modulo m: Ar Br, Ai Bi, (Ar + Ai)(Br + Bi)."""
    return tuple(sym(_exact_matmul(a, b), m) for a, b in zip(A3, B3))


def post_3m(P1, P2, P3, m: int):
    """Eq. (1): C = (P1 - P2) + i (P3 - P1 - P2) (mod m)."""
    return sym(P1 - P2, m), sym(P3 - P1 - P2, m)


# ----------------------------------------------------------------------------- CRT (Section 3.1, Algorithm 1 steps 5-6)
def product(moduli):
    M = 1
    for q in moduli:
        M *= int(q)
    return M


def crt(residues, moduli):
    """X = ( sum_l ((x_l q_l) mod m_l) (M/m_l) ) mod M with q_l = (M/m_l mod m_l)^-1 mod m_l, in [0, M)."""
    M = product(moduli)
    acc = 0
    for x, ml in zip(residues, moduli):
        ml = int(ml)
        Wl = M // ml
        ql = pow(Wl % ml, -1, ml)
        x = np.asarray(x).astype(object) if isinstance(x, np.ndarray) else int(x)
        acc = acc + ((x * ql) % ml) * Wl
    return acc % M


def lift(X, M: int):
    """Algorithm 1 step 6: representative in [-M/2, M/2); for odd M this is [-(M-1)/2, (M-1)/2]."""
    h = M // 2
    return (X + h) % M - h


# ----------------------------------------------------------------------------- scaling (Algorithm 1 steps 2, 3, 7)
def scaling_targets(M: int, k: int, herk: bool = False):
    """P_t = floor(log2((M-1)/2)); the row budget P_A and column budget P_B split it (equal for HERK);
    c_k = ceil(log2(2k)/2) accounts for the 2k real terms of a row's 2-norm."""
    Pt = ((M - 1) // 2).bit_length() - 1
    PA, PB = -((-Pt) // 2), Pt // 2
    if herk:
        PA = PB = Pt // 2
    ck = 0
    while 4 ** ck < 2 * max(k, 1):
        ck += 1
    return Pt, PA, PB, ck


def scaling_exponents(Z, axis: int, P: int, ck: int):
    """sigma_i = 2^e_i (axis=1: per row of A) or tau_j = 2^f_j (axis=0: per column of B).
    mu = largest |Re| or |Im| in the row/column, x = floor(log2 mu), e = x + 1 + c_k - P; zero rows get e = 0.
    Then |z'| <= |z| 2^-e < 2^(P - c_k), so the row's 2-norm is at most sqrt(2k) 2^(P-c_k) <= 2^P."""
    Z = np.asarray(Z)
    mags = np.maximum(np.abs(Z.real), np.abs(Z.imag)).astype(np.float64)
    mu = mags.max(axis=axis, initial=0.0)
    _, ex = np.frexp(mu)                       # mu = f 2^ex with 0.5 <= f < 1, so floor(log2 mu) = ex - 1
    e = ex.astype(np.int64) + ck - P
    return np.where(mu > 0, e, 0).astype(np.int64)


TIGHT_FRAC_BITS = 20      # resolution of the fixed-point magnitudes of the 2-norm scaling rule


def scaling_exponents_2norm(Z, axis: int, P: int):
    """The tighter choice of sigma / tau the paper points to the literature for (Algorithm 1 step 2): bound the row's
    2-norm itself instead of sqrt(2k) times its largest part.  All-integer so that it is reproducible bit for bit:
    with mu, x as in `scaling_exponents`, every part v of the row is rounded UP to the fixed-point magnitude
    u = ceil(|v| 2^(20 - (x+1))) (an integer <= 2^20), Q = sum u^2 over the 2k parts, t = the smallest integer with
    4^t >= Q, and e = x + 1 - P + (t - 20).  Then |v| <= u 2^(x+1-20), so the row's 2-norm is at most
    2^(x+1-20) sqrt(Q) <= 2^(x+1-20+t) = 2^(P+e): the scaled row has 2-norm <= 2^P, which is all the overflow proof needs.
    The largest part has u >= 2^19, so t >= 19; and Q <= 2k 4^20, so t - 20 <= c_k: the exponent is never above the
    max-based rule's."""
    from fractions import Fraction
    Z = np.asarray(Z)
    if axis == 0:
        Z = Z.T
    rows = Z.shape[0]
    e = np.zeros(rows, dtype=np.int64)
    for i in range(rows):
        parts = np.concatenate([np.abs(Z[i].real), np.abs(Z[i].imag)]).astype(np.float64)
        mu = parts.max(initial=0.0)
        if not mu > 0:
            continue
        x = int(np.frexp(mu)[1]) - 1
        scale = Fraction(2) ** (TIGHT_FRAC_BITS - (x + 1))
        Q = 0
        for v in parts:
            if v != 0:
                f = Fraction(float(v)) * scale
                u = -((-f.numerator) // f.denominator)          # ceil
                Q += u * u
        t = 0
        while 4 ** t < Q:
            t += 1
        e[i] = x + 1 - P + (t - TIGHT_FRAC_BITS)
    return e


def _quantise_part(x, e, int64_ok: bool = False):
    """trunc(x 2^-e) exactly, elementwise; x float array, e broadcastable integer array.  Object array of ints
    (int64_ok: an int64 array instead when no entry needs a left shift -- the same values, for large inputs)."""
    x = np.asarray(x, dtype=np.float64)
    mant, ex = np.frexp(x)
    Mi = np.ldexp(mant, 53).astype(np.int64)             # x = Mi 2^(ex-53), |Mi| < 2^53, exact
    sh = ex.astype(np.int64) - 53 - e                    # x 2^-e = Mi 2^sh
    sgn = np.sign(Mi)
    mag = np.abs(Mi)
    right = np.minimum(np.maximum(-sh, 0), 63)
    out = sgn * (mag >> right)                           # truncation toward zero on the magnitude
    pos = sh > 0
    if not (int64_ok and not np.any(pos)):
        out = out.astype(object)
    if np.any(pos):                                      # left shifts: the value may not fit 64 bits
        flat_out = out.ravel()
        flat_M = Mi.ravel()
        flat_sh = np.broadcast_to(sh, x.shape).ravel()
        for idx in np.flatnonzero(pos.ravel()):
            flat_out[idx] = int(flat_M[idx]) << int(flat_sh[idx])
        out = flat_out.reshape(x.shape)
    return out


def quantise(Z, e, axis: int, int64_ok: bool = False):
    """Algorithm 1 step 3 with truncation: (Zr', Zi') = trunc(parts of Z / 2^e) with e per row (axis=1) or column (axis=0)."""
    Z = np.asarray(Z)
    eb = e[:, None] if axis == 1 else e[None, :]
    return _quantise_part(Z.real, eb, int64_ok), _quantise_part(Z.imag, eb, int64_ok)


def round_int_nearest_even(X: int, bits: int):
    """X ~ Y 2^t with |Y| <= 2^bits, round-to-nearest-even once."""
    a = abs(X)
    n = a.bit_length()
    if n <= bits:
        return X, 0
    t = n - bits
    q, r = divmod(a, 1 << t)
    half = 1 << (t - 1)
    if r > half or (r == half and (q & 1)):
        q += 1
    return (q if X >= 0 else -q), t


def unscale(X, e_row, f_col, bits: int = 53):
    """Algorithm 1 step 7: c_ij sigma_i tau_j with one rounding of the integer to `bits` significant bits."""
    m, n = X.shape
    out = np.zeros((m, n), dtype=np.float64)
    for i in range(m):
        for j in range(n):
            y, t = round_int_nearest_even(int(X[i, j]), bits)
            out[i, j] = math.ldexp(float(y), t + int(e_row[i]) + int(f_col[j]))
    return out


def _small(a):
    """Object array of ints -> int64 when it fits (faster residues)."""
    if a.size == 0:
        return a.astype(np.int64)
    mx = max(abs(int(a.max())), abs(int(a.min())))
    return a.astype(np.int64) if mx < 2 ** 62 else a


def _residue_planes(Zr, Zi, moduli, roots):
    """Per modulus: (X+, X-) for a 2M modulus (root given), (Xr, Xi, Xr + Xi) for a 3M modulus (root None)."""
    Zr, Zi = _small(Zr), _small(Zi)
    planes = []
    for ml, sl in zip(moduli, roots):
        # reduce first so that s * Zi stays small in int64
        zr = Zr % ml
        zi = Zi % ml
        pl = pre_2m(zr, zi, ml, sl) if sl is not None else pre_3m(zr, zi, ml)
        planes.append(tuple(np.asarray(p).astype(np.int64) for p in pl))
    return planes


def roots_of(moduli):
    """s_l for the 2M moduli, None for the others (they take 3M multiplication)."""
    return [sqrt_minus_one(q) if is_2m_modulus(q) else None for q in moduli]


def _multiply_and_post(Apl, Bpl, moduli, roots):
    Cpm, res_r, res_i = [], [], []
    for Ap, Bp, ml, sl in zip(Apl, Bpl, moduli, roots):
        if sl is not None:
            Cp, Cm = mul_2m(Ap[0], Bp[0], ml), mul_2m(Ap[1], Bp[1], ml)   # (2b)
            Cpm.append((Cp, Cm))
            r, i = post_2m(Cp, Cm, ml, sl)                                 # (2c)
        else:
            P = mul_3m(Ap, Bp, ml)                                         # Eq. (1) modulo m
            Cpm.append(P)
            r, i = post_3m(P[0], P[1], P[2], ml)
        res_r.append(r)
        res_i.append(i)
    return Cpm, res_r, res_i


# ----------------------------------------------------------------------------- whole paths
def gemm2m_int_staged(Ar, Ai, Br, Bi, nmod: int):
    """Integer 2M multiplication (Section 2; 3M for the non-2M moduli beyond the 22nd) + CRT over the first `nmod` moduli.
    Returns a dict of stages."""
    moduli = hybrid_moduli(nmod)
    roots = roots_of(moduli)
    M = product(moduli)
    Ar, Ai, Br, Bi = (np.asarray(x).astype(object) for x in (Ar, Ai, Br, Bi))
    Apl = _residue_planes(Ar, Ai, moduli, roots)
    Bpl = _residue_planes(Br, Bi, moduli, roots)
    Cpm, res_r, res_i = _multiply_and_post(Apl, Bpl, moduli, roots)
    Xr, Xi = lift(crt(res_r, moduli), M), lift(crt(res_i, moduli), M)
    return dict(moduli=moduli, roots=roots, M=M, Apm=Apl, Bpm=Bpl, Cpm=Cpm, res_r=res_r, res_i=res_i, Xr=Xr, Xi=Xi)


def zgemm2m_staged(A, B, nmod: int, herk: bool = False, out_bits: int = 53, upto: str = "all", scaling: str = "max"):
    """Algorithm 1 on floating-point A (m x k), B (k x n).  For herk=True pass B = A^H.
    upto = "pre" stops after the residue planes (cheap at large sizes).  scaling = "max" (largest part times sqrt(2k))
    or "2norm" (`scaling_exponents_2norm`)."""
    A = np.asarray(A)
    B = np.asarray(B)
    k = A.shape[1]
    moduli = hybrid_moduli(nmod)                                   # step 1 (2M moduli only while nmod <= 22)
    roots = roots_of(moduli)
    M = product(moduli)
    Pt, PA, PB, ck = scaling_targets(M, k, herk)
    if scaling == "2norm":
        eA = scaling_exponents_2norm(A, 1, PA)                     # step 2
        eB = scaling_exponents_2norm(B, 0, PB)
    else:
        eA = scaling_exponents(A, 1, PA, ck)
        eB = scaling_exponents(B, 0, PB, ck)
    Aq = quantise(A, eA, 1)                                        # step 3
    Bq = quantise(B, eB, 0)
    Apl = _residue_planes(Aq[0], Aq[1], moduli, roots)             # step 4: (2a), or the 3M sums
    Bpl = _residue_planes(Bq[0], Bq[1], moduli, roots)
    st = dict(moduli=moduli, roots=roots, M=M, Pt=Pt, PA=PA, PB=PB, ck=ck, eA=eA, eB=eB, Aq=Aq, Bq=Bq,
              Apm=Apl, Bpm=Bpl)
    if upto == "pre":
        return st
    Cpm, res_r, res_i = _multiply_and_post(Apl, Bpl, moduli, roots)      # (2b), (2c) / Eq. (1)
    Xr, Xi = lift(crt(res_r, moduli), M), lift(crt(res_i, moduli), M)   # steps 5, 6
    C = unscale(Xr, eA, eB, out_bits) + 1j * unscale(Xi, eA, eB, out_bits)   # step 7
    st.update(Cpm=Cpm, res_r=res_r, res_i=res_i, Xr=Xr, Xi=Xi, C=C)
    return st


def scaling_targets_real(M: int, k: int):
    """Real scheme: a row has k real terms, so c_k = ceil(log2(k)/2); P_t, P_A, P_B as in `scaling_targets`."""
    Pt = ((M - 1) // 2).bit_length() - 1
    ck = 0
    while 4 ** ck < max(k, 1):
        ck += 1
    return Pt, -((-Pt) // 2), Pt // 2, ck


def dgemm_o2_staged(A, B, nmod: int, out_bits: int = 53):
    """Section 3.1: the real Ozaki-II scheme C = A B for real A (m x k), B (k x n): scale and truncate, one real integer
    GEMM per modulus of the real set, CRT, lift, unscale.  The same readings as for Algorithm 1 (power-of-two scale
    factors from the largest magnitude of a row times sqrt(k), truncation, symmetric residues, single rounding)."""
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    k = A.shape[1]
    moduli = greedy_real_moduli()[:nmod]
    M = product(moduli)
    Pt, PA, PB, ck = scaling_targets_real(M, k)
    eA = scaling_exponents(A + 0j, 1, PA, ck)
    eB = scaling_exponents(B + 0j, 0, PB, ck)
    Aq = _quantise_part(A, eA[:, None])
    Bq = _quantise_part(B, eB[None, :])
    Apl = [np.asarray(sym(_small(Aq) % ml, ml)).astype(np.int64) for ml in moduli]
    Bpl = [np.asarray(sym(_small(Bq) % ml, ml)).astype(np.int64) for ml in moduli]
    Cpl = [sym(_exact_matmul(a, b_), ml) for a, b_, ml in zip(Apl, Bpl, moduli)]
    X = lift(crt(Cpl, moduli), M)
    C = unscale(X, eA, eB, out_bits)
    return dict(moduli=moduli, M=M, Pt=Pt, PA=PA, PB=PB, ck=ck, eA=eA, eB=eB, Aq=Aq, Bq=Bq, Apl=Apl, Bpl=Bpl, Cpl=Cpl, X=X, C=C)


def syrk_complexify(X):
    """Section 5, SYRK paragraph: split real X (n x k) evenly in the k dimension, X = [X1 | X2] (a zero column is appended
    when k is odd), and form Z = X1 + i X2; then X X^T = Re(Z Z^H)."""
    X = np.asarray(X, dtype=np.float64)
    n, k = X.shape
    k2 = (k + 1) // 2
    Z = np.zeros((n, k2), dtype=np.complex128, order="F")
    Z.real = X[:, :k2]
    Z.imag[:, : k - k2] = X[:, k2:]
    return Z


def zher2k2m_staged(A, B, nmod: int, out_bits: int = 53):
    """Section 5, HER2K with 2M Ozaki-II: one scale vector for A and B (sigma = tau), then per modulus
    C+ = A+ B-^T + B+ A-^T and C- = A- B+^T + B- A+^T (mod m), Eq. (2c), CRT, lift, unscale."""
    A = np.asarray(A)
    B = np.asarray(B)
    n, k = A.shape
    moduli = greedy_2m_moduli()[:nmod]
    roots = [sqrt_minus_one(q) for q in moduli]
    M = product(moduli)
    Pt, P, _, ck = scaling_targets(M, 2 * k, herk=True)     # an entry is an inner product of rows of 2k complex numbers
    eA = scaling_exponents(np.concatenate([A, B], axis=1), 1, P, ck)
    Aq, Bq = quantise(A, eA, 1), quantise(B, eA, 1)
    Apl = _residue_planes(Aq[0], Aq[1], moduli, roots)
    Bpl = _residue_planes(Bq[0], Bq[1], moduli, roots)
    Cpm, res_r, res_i = [], [], []
    for (Ap, Am), (Bp, Bm), ml, sl in zip(Apl, Bpl, moduli, roots):
        Cp = sym(_exact_matmul(Ap, Bm.T) + _exact_matmul(Bp, Am.T), ml)
        Cm = sym(_exact_matmul(Am, Bp.T) + _exact_matmul(Bm, Ap.T), ml)
        Cpm.append((Cp, Cm))
        r, i = post_2m(Cp, Cm, ml, sl)
        res_r.append(r)
        res_i.append(i)
    Xr, Xi = lift(crt(res_r, moduli), M), lift(crt(res_i, moduli), M)
    C = unscale(Xr, eA, eA, out_bits) + 1j * unscale(Xi, eA, eA, out_bits)
    return dict(moduli=moduli, roots=roots, M=M, Pt=Pt, P=P, ck=ck, eA=eA, Aq=Aq, Bq=Bq, Apm=Apl, Bpm=Bpl, Cpm=Cpm,
                Xr=Xr, Xi=Xi, C=C)


def staged_samples(st, pairs, out_bits: int = 53):
    """Exact lifted integers and final values for sampled entries, from the quantised matrices of a
    `zgemm2m_staged(..., upto="pre")` result: the 4M product of the quantised Gaussian integers reduced
    mod M -- the value steps 4-6 must reproduce whatever multiplication method is used (Section 6)."""
    M = st["M"]
    Ar, Ai = st["Aq"]
    Br, Bi = st["Bq"]
    vals = np.zeros(len(pairs), dtype=np.complex128)
    Xs = []
    for t, (i, j) in enumerate(np.asarray(pairs).tolist()):
        ar = [int(v) for v in Ar[i, :]]
        ai = [int(v) for v in Ai[i, :]]
        br = [int(v) for v in Br[:, j]]
        bi = [int(v) for v in Bi[:, j]]
        cr = sum(x * y for x, y in zip(ar, br)) - sum(x * y for x, y in zip(ai, bi))
        ci = sum(x * y for x, y in zip(ar, bi)) + sum(x * y for x, y in zip(ai, br))
        xr, xi = lift(cr, M), lift(ci, M)
        Xs.append((xr, xi))
        sc = int(st["eA"][i]) + int(st["eB"][j])
        yr, tr = round_int_nearest_even(xr, out_bits)
        yi, ti = round_int_nearest_even(xi, out_bits)
        vals[t] = complex(math.ldexp(float(yr), tr + sc), math.ldexp(float(yi), ti + sc))
    return Xs, vals

"""The plain 4M definitions -- TEST INFRASTRUCTURE ONLY (see the package docstring).

  gauss4m_exact      exact Gaussian-integer product (Section 1: C = (ArBr - AiBi) + i(ArBi + AiBr)),
                     __int128 accumulation in C, returned as Python integers.
  gauss4m_python     the same in pure Python integers (tiny cases; pins the C routine).
  symmetric_residue  representative of x mod M in [-(M-1)/2, (M-1)/2] (Section 2, first paragraph;
                     Algorithm 1 step 6).
  zgemm4m_dd         4M complex product with double-double accumulation plus D = |A||B|.
  zherk_dd, zher2k_dd, dsyrk_dd, dsyr2k_dd   the rank-k definitions of Section 5 (C = A A^H, A B^H + B A^H, A A^T,
                     A B^T + B A^T), each entry one double-double accumulation.
  componentwise_error  max_ij |C - Cref| / D_ij, the acceptance metric.
"""
from __future__ import annotations

import ctypes

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i64(x):
    return ctypes.c_int64(int(x))


def gauss4m_exact(Ar, Ai, Br, Bi):
    """Exact C_r, C_i (object arrays of Python ints) for integer matrices; requires |entries| < 2^62 and
    results < 2^127 (true whenever k * max|a| * max|b| * 2 < 2^127)."""
    Ar, Ai, Br, Bi = (np.asfortranarray(x, dtype=np.int64) for x in (Ar, Ai, Br, Bi))
    m, k = Ar.shape
    k2, n = Br.shape
    assert k == k2 and Ai.shape == Ar.shape and Bi.shape == Br.shape
    amax = max(int(np.abs(Ar).max(initial=0)), int(np.abs(Ai).max(initial=0)))
    bmax = max(int(np.abs(Br).max(initial=0)), int(np.abs(Bi).max(initial=0)))
    assert 2 * max(k, 1) * amax * bmax < 2 ** 127, "result would overflow __int128"
    outs = [np.zeros((m, n), dtype=dt, order="F") for dt in (np.int64, np.uint64, np.int64, np.uint64)]
    if m and n:
        lib().oracle_gauss4m_i128(_i64(m), _i64(n), _i64(k), _p(Ar), _p(Ai), _i64(max(m, 1)),
                                  _p(Br), _p(Bi), _i64(max(k, 1)), _p(outs[0]), _p(outs[1]), _p(outs[2]),
                                  _p(outs[3]), _i64(max(m, 1)))
    cr = outs[0].astype(object) * (1 << 64) + outs[1].astype(object)
    ci = outs[2].astype(object) * (1 << 64) + outs[3].astype(object)
    return cr, ci


def gauss4m_python(Ar, Ai, Br, Bi):
    """Pure-Python-integer 4M product (tiny cases only)."""
    m, k = np.shape(Ar)
    n = np.shape(Br)[1]
    cr = np.zeros((m, n), dtype=object)
    ci = np.zeros((m, n), dtype=object)
    for i in range(m):
        for j in range(n):
            r = 0
            im = 0
            for p in range(k):
                ar, ai, br, bi = int(Ar[i][p]), int(Ai[i][p]), int(Br[p][j]), int(Bi[p][j])
                r += ar * br - ai * bi
                im += ar * bi + ai * br
            cr[i, j] = r
            ci[i, j] = im
    return cr, ci


def symmetric_residue(x, M):
    """x mod M as the representative in [-(M-1)/2, (M-1)/2]; M odd.  Works on ints and object arrays."""
    assert M % 2 == 1
    h = (M - 1) // 2
    return (x + h) % M - h


def gauss4m_mod(Ar, Ai, Br, Bi, M):
    """What gemm2m_gaussian_int must return: the exact 4M product reduced to the symmetric residue mod M,
    as int64 arrays (M < 2^63)."""
    cr, ci = gauss4m_exact(Ar, Ai, Br, Bi)
    return (np.asfortranarray(symmetric_residue(cr, M).astype(np.int64)),
            np.asfortranarray(symmetric_residue(ci, M).astype(np.int64)))


def _as_z(A):
    A = np.asarray(A)
    if A.dtype == np.complex64:       # widen exactly
        A = A.astype(np.complex128)
    return np.asfortranarray(A, dtype=np.complex128)


def zgemm4m_dd(A, B):
    """C (complex128, each part a double-double 4M dot product rounded once) and D = |A||B| (float64)."""
    A, B = _as_z(A), _as_z(B)
    m, k = A.shape
    k2, n = B.shape
    assert k == k2
    C = np.zeros((m, n), dtype=np.complex128, order="F")
    D = np.zeros((m, n), dtype=np.float64, order="F")
    if m and n:
        lib().oracle_zgemm4m_dd(_i64(m), _i64(n), _i64(k), _p(A), _i64(max(m, 1)), _p(B), _i64(max(k, 1)),
                                _p(C), _i64(max(m, 1)), _p(D), _i64(max(m, 1)))
    return C, D


def zgemm4m_dd_samples(A, B, pairs):
    """The same for sampled entries; `pairs` is an (S, 2) int array of (row, column)."""
    A, B = _as_z(A), _as_z(B)
    m, k = A.shape
    pairs = np.ascontiguousarray(pairs, dtype=np.int64)
    rows = np.ascontiguousarray(pairs[:, 0])
    cols = np.ascontiguousarray(pairs[:, 1])
    S = rows.shape[0]
    C = np.zeros(S, dtype=np.complex128)
    D = np.zeros(S, dtype=np.float64)
    if S:
        lib().oracle_zgemm4m_dd_samples(_i64(k), _p(A), _i64(max(m, 1)), _p(B), _i64(max(k, 1)), _i64(S),
                                        _p(rows), _p(cols), _p(C), _p(D))
    return C, D


def zgemm4m_dd2(A1, B1, A2, B2):
    """C = A1 B1 + A2 B2 accumulated in double-double over both products, and D = |A1||B1| + |A2||B2|."""
    A1, B1, A2, B2 = _as_z(A1), _as_z(B1), _as_z(A2), _as_z(B2)
    m, k = A1.shape
    n = B1.shape[1]
    assert A2.shape == (m, k) and B1.shape == (k, n) and B2.shape == (k, n)
    C = np.zeros((m, n), dtype=np.complex128, order="F")
    D = np.zeros((m, n), dtype=np.float64, order="F")
    if m and n:
        lib().oracle_zgemm4m_dd2(_i64(m), _i64(n), _i64(k), _p(A1), _i64(max(m, 1)), _p(B1), _i64(max(k, 1)),
                                 _p(A2), _i64(max(m, 1)), _p(B2), _i64(max(k, 1)), _p(C), _i64(max(m, 1)), _p(D), _i64(max(m, 1)))
    return C, D


def apply_op(X, trans):
    """op(X) of the BLAS interface: 'N' -> X, 'T' -> X^T, 'C' -> X^H."""
    X = np.asarray(X)
    t = trans.upper()
    if t == "N":
        return X
    if t == "T":
        return X.T
    if t == "C":
        return X.conj().T
    raise ValueError(trans)


def zgemm_ex_dd(transa, transb, alpha, A, B, beta, C0):
    """The ZGEMM definition alpha op(A) op(B) + beta C0 (the paper's Section 6 fixes alpha = 1, beta = 0, no transposes;
    this is the BLAS convention beyond that).  The product is the double-double 4M product rounded once; the combination
    with alpha, beta is evaluated in extended precision (64-bit significand) and rounded once.
    Returns the result and the error scale D = |alpha| |op(A)||op(B)| + |beta| |C0|."""
    alpha, beta = complex(alpha), complex(beta)
    L = np.longdouble
    opA, opB = apply_op(A, transa), apply_op(B, transb)
    shape = (opA.shape[0], opB.shape[1])
    re, im, scale = np.zeros(shape, dtype=L), np.zeros(shape, dtype=L), np.zeros(shape)
    if alpha != 0:                      # alpha = 0: A and B are not referenced
        P, D = zgemm4m_dd(opA, opB)
        pr, pi = P.real.astype(L), P.imag.astype(L)
        re = L(alpha.real) * pr - L(alpha.imag) * pi
        im = L(alpha.real) * pi + L(alpha.imag) * pr
        scale = abs(alpha) * D
    if beta != 0:                       # beta = 0: C0 is not referenced (it may hold NaNs)
        C0 = _as_z(C0)
        cr, ci = C0.real.astype(L), C0.imag.astype(L)
        re = re + L(beta.real) * cr - L(beta.imag) * ci
        im = im + L(beta.real) * ci + L(beta.imag) * cr
        scale = scale + abs(beta) * np.abs(C0)
    return np.asfortranarray(re.astype(np.float64) + 1j * im.astype(np.float64)), np.asfortranarray(scale)


def zherk_dd(A):
    """Section 5, HERK: C = A A^H."""
    A = _as_z(A)
    return zgemm4m_dd(A, A.conj().T)


def zher2k_dd(A, B):
    """Section 5, HER2K: C = A B^H + B A^H."""
    A, B = _as_z(A), _as_z(B)
    return zgemm4m_dd2(A, B.conj().T, B, A.conj().T)


def dgemm_dd(A, B):
    """Real C = A B with every dot product in double-double, rounded once, and D = |A||B|."""
    A, B = np.asarray(A, dtype=np.float64), np.asarray(B, dtype=np.float64)
    C, D = zgemm4m_dd(A.astype(np.complex128), B.astype(np.complex128))
    return np.asfortranarray(C.real), D


def dsyrk_dd(A):
    """Section 5, SYRK: C = A A^T for real A (returned real)."""
    A = np.asarray(A, dtype=np.float64)
    C, D = zgemm4m_dd(A.astype(np.complex128), A.T.astype(np.complex128))
    return np.asfortranarray(C.real), D


def dsyr2k_dd(A, B):
    """Section 5, SYR2K: C = A B^T + B A^T for real A, B (returned real)."""
    A, B = np.asarray(A, dtype=np.float64), np.asarray(B, dtype=np.float64)
    C, D = zgemm4m_dd2(A.astype(np.complex128), B.T.astype(np.complex128), B.astype(np.complex128), A.T.astype(np.complex128))
    return np.asfortranarray(C.real), D


def componentwise_error(C, Cref, D):
    """max_ij |C_ij - Cref_ij| / D_ij, skipping entries with D_ij = 0 (those must match exactly)."""
    C = np.asarray(C, dtype=np.complex128)
    diff = np.abs(C - Cref)
    nz = D > 0
    if np.any(~nz) and np.any(diff[~nz] != 0):
        return np.inf
    if not np.any(nz):
        return 0.0
    return float(np.max(diff[nz] / D[nz]))

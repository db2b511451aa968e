"""Seeded synthetic input generators shared by the tests, the benchmark and the oracle checks.

This module holds none of the method's arithmetic: it only draws random matrices with the
shapes and value distributions of the workloads (Section 6 of the paper uses synthetic
random matrices; its accuracy test uses the "(rand-0.5)*exp(phi*randn)" distribution with
phi = 0.5).  Draw order is always A_r, A_i, B_r, B_i, each as one full matrix, from
``numpy.random.default_rng(seed)``.  All matrices are returned column-major (Fortran
order), complex ones as numpy complex arrays whose memory is interleaved (re, im).
"""
from __future__ import annotations

import numpy as np


def _part(rng, rows, cols, dist, phi):
    if dist == "uniform":            # parts uniform in (-1, 1)
        return rng.uniform(-1.0, 1.0, size=(rows, cols))
    if dist == "phi":                # (rand - 0.5) * exp(phi * randn): exponent spread grows with phi
        u = rng.random(size=(rows, cols))
        g = rng.standard_normal(size=(rows, cols))
        return (u - 0.5) * np.exp(phi * g)
    raise ValueError(f"unknown distribution {dist!r}")


def _complex_f(re, im, dtype):
    out = np.empty(re.shape, dtype=dtype, order="F")
    out.real = re
    out.imag = im
    return out


def gaussian_int_inputs(m, n, k, seed, lo=-16, hi=16):
    """Four int8 matrices A_r, A_i (m x k) and B_r, B_i (k x n), entries uniform integers in [lo, hi]."""
    rng = np.random.default_rng(seed)
    mats = []
    for rows, cols in ((m, k), (m, k), (k, n), (k, n)):
        mats.append(np.asfortranarray(rng.integers(lo, hi + 1, size=(rows, cols), dtype=np.int64).astype(np.int8)))
    return tuple(mats)


def complex_inputs(m, n, k, seed, dist="uniform", phi=0.5, dtype=np.complex128):
    """A (m x k) and B (k x n), column-major complex; parts drawn from `dist` ("uniform" or "phi")."""
    rng = np.random.default_rng(seed)
    ar = _part(rng, m, k, dist, phi)
    ai = _part(rng, m, k, dist, phi)
    br = _part(rng, k, n, dist, phi)
    bi = _part(rng, k, n, dist, phi)
    return _complex_f(ar, ai, dtype), _complex_f(br, bi, dtype)


def herk_input(n, k, seed, dist="uniform", phi=0.5, dtype=np.complex128):
    """A (n x k), column-major complex, for the rank-k update C = A A^H."""
    rng = np.random.default_rng(seed)
    ar = _part(rng, n, k, dist, phi)
    ai = _part(rng, n, k, dist, phi)
    return _complex_f(ar, ai, dtype)


def sample_indices(m, n, count, seed, tile=128):
    """Row/column index pairs for sampled checks at large sizes: random entries plus the first and
    last rows/columns and the indices next to tile edges."""
    rng = np.random.default_rng(seed)
    special_r = sorted({i for i in (0, 1, tile - 1, tile, 2 * tile - 1, 2 * tile, m - 2, m - 1) if 0 <= i < m})
    special_c = sorted({j for j in (0, 1, tile - 1, tile, 2 * tile - 1, 2 * tile, n - 2, n - 1) if 0 <= j < n})
    pairs = [(i, j) for i in special_r for j in special_c]
    extra = max(0, count - len(pairs))
    ri = rng.integers(0, m, size=extra)
    ci = rng.integers(0, n, size=extra)
    pairs += list(zip(ri.tolist(), ci.tolist()))
    return np.array(pairs, dtype=np.int64)

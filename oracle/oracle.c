/*
 * CPU oracle for complex matrix products -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, obviously-correct statements of what the 2M / Ozaki-II path must compute.
 * Nothing here is used by the GPU library; only tests, the smoke check and the benchmark's
 * cpu_baseline leg call it.  It shares no code, table or constant with the CUDA path.
 *
 *   oracle_gauss4m_i128 : the 4M definition C = (ArBr - AiBi) + i(ArBi + AiBr) over the
 *                         integers (Section 1 of the paper), accumulated in __int128.
 *   oracle_zgemm4m_dd   : the same 4M definition on floating-point data, each of the four
 *                         real dot products accumulated in double-double (about 106 bits),
 *                         rounded once to double; also D = |A||B| with complex moduli.
 *   oracle_zgemm4m_dd_samples : the same for a list of (i, j) entries only.
 *   oracle_zgemm4m_dd2  : C = A1 B1 + A2 B2 (the two-product sums of the rank-2k updates of Section 5), one double-double
 *                         accumulation over both products, rounded once.
 *
 * All matrices are column-major; complex matrices are interleaved (re, im) doubles with the
 * leading dimension counted in complex elements.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef __int128 i128;

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* 4M integer product, Section 1: C_r = A_r B_r - A_i B_i, C_i = A_r B_i + A_i B_r.
 * Inputs int64 (col-major, lda/ldb in elements), outputs split into high (signed) and low
 * (unsigned) 64-bit halves of the exact 128-bit result. */
void oracle_gauss4m_i128(int64_t m, int64_t n, int64_t k,
                         const int64_t* Ar, const int64_t* Ai, int64_t lda,
                         const int64_t* Br, const int64_t* Bi, int64_t ldb,
                         int64_t* Cr_hi, uint64_t* Cr_lo, int64_t* Ci_hi, uint64_t* Ci_lo, int64_t ldc) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n; ++j) {
        for (int64_t i = 0; i < m; ++i) {
            i128 rr = 0, ii = 0, ri = 0, ir = 0;
            for (int64_t p = 0; p < k; ++p) {
                i128 ar = Ar[i + p * lda], ai = Ai[i + p * lda];
                i128 br = Br[p + j * ldb], bi = Bi[p + j * ldb];
                rr += ar * br;
                ii += ai * bi;
                ri += ar * bi;
                ir += ai * br;
            }
            i128 cr = rr - ii, ci = ri + ir;
            Cr_hi[i + j * ldc] = (int64_t)(cr >> 64);
            Cr_lo[i + j * ldc] = (uint64_t)cr;
            Ci_hi[i + j * ldc] = (int64_t)(ci >> 64);
            Ci_lo[i + j * ldc] = (uint64_t)ci;
        }
    }
}

/* ---- double-double helpers (error-free transformations) ---- */
typedef struct { double hi, lo; } dd;

static inline dd dd_two_sum(double a, double b) {
    double s = a + b;
    double bb = s - a;
    double e = (a - (s - bb)) + (b - bb);
    dd r = {s, e};
    return r;
}
static inline dd dd_two_prod(double a, double b) {
    double p = a * b;
    double e = fma(a, b, -p);
    dd r = {p, e};
    return r;
}
/* acc += a*b, acc in double-double */
static inline dd dd_mac(dd acc, double a, double b) {
    dd p = dd_two_prod(a, b);
    dd s = dd_two_sum(acc.hi, p.hi);
    double lo = s.lo + (acc.lo + p.lo);
    dd r = dd_two_sum(s.hi, lo);
    return r;
}
static inline dd dd_add(dd a, dd b) {
    dd s = dd_two_sum(a.hi, b.hi);
    double lo = s.lo + (a.lo + b.lo);
    return dd_two_sum(s.hi, lo);
}
static inline dd dd_neg(dd a) { dd r = {-a.hi, -a.lo}; return r; }

static void entry_dd(int64_t k, const double* arow /* k interleaved */, const double* bcol /* k interleaved */,
                     double* cr, double* ci, double* dabs) {
    dd rr = {0, 0}, ii = {0, 0}, ri = {0, 0}, ir = {0, 0};
    double d = 0.0;
    for (int64_t p = 0; p < k; ++p) {
        double ar = arow[2 * p], ai = arow[2 * p + 1];
        double br = bcol[2 * p], bi = bcol[2 * p + 1];
        rr = dd_mac(rr, ar, br);
        ii = dd_mac(ii, ai, bi);
        ri = dd_mac(ri, ar, bi);
        ir = dd_mac(ir, ai, br);
        d += hypot(ar, ai) * hypot(br, bi);
    }
    dd r = dd_add(rr, dd_neg(ii));
    dd i = dd_add(ri, ir);
    *cr = r.hi + r.lo;
    *ci = i.hi + i.lo;
    *dabs = d;
}

/* 4M floating-point product in double-double, Section 1; D = |A||B| (entrywise complex moduli). */
void oracle_zgemm4m_dd(int64_t m, int64_t n, int64_t k,
                       const double* A, int64_t lda, const double* B, int64_t ldb,
                       double* C, int64_t ldc, double* D, int64_t ldd) {
#pragma omp parallel
    {
        double* arow = (double*)malloc(sizeof(double) * 2 * (size_t)(k > 0 ? k : 1));
#pragma omp for schedule(static)
        for (int64_t i = 0; i < m; ++i) {
            for (int64_t p = 0; p < k; ++p) {          /* gather row i of column-major A */
                arow[2 * p] = A[2 * (i + p * lda)];
                arow[2 * p + 1] = A[2 * (i + p * lda) + 1];
            }
            for (int64_t j = 0; j < n; ++j) {
                double cr, ci, d;
                entry_dd(k, arow, B + 2 * j * ldb, &cr, &ci, &d);
                C[2 * (i + j * ldc)] = cr;
                C[2 * (i + j * ldc) + 1] = ci;
                D[i + j * ldd] = d;
            }
        }
        free(arow);
    }
}

/* The same for `count` sampled entries (rows[s], cols[s]); outputs C (interleaved) and D of length count. */
void oracle_zgemm4m_dd_samples(int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb,
                               int64_t count, const int64_t* rows, const int64_t* cols,
                               double* C, double* D) {
#pragma omp parallel
    {
        double* arow = (double*)malloc(sizeof(double) * 2 * (size_t)(k > 0 ? k : 1));
#pragma omp for schedule(dynamic, 16)
        for (int64_t s = 0; s < count; ++s) {
            int64_t i = rows[s], j = cols[s];
            for (int64_t p = 0; p < k; ++p) {
                arow[2 * p] = A[2 * (i + p * lda)];
                arow[2 * p + 1] = A[2 * (i + p * lda) + 1];
            }
            double cr, ci, d;
            entry_dd(k, arow, B + 2 * j * ldb, &cr, &ci, &d);
            C[2 * s] = cr;
            C[2 * s + 1] = ci;
            D[s] = d;
        }
        free(arow);
    }
}

/* C = A1 B1 + A2 B2 with A1, A2: m x k and B1, B2: k x n (all interleaved complex, column-major); D = |A1||B1| + |A2||B2|. */
void oracle_zgemm4m_dd2(int64_t m, int64_t n, int64_t k,
                        const double* A1, int64_t lda1, const double* B1, int64_t ldb1,
                        const double* A2, int64_t lda2, const double* B2, int64_t ldb2,
                        double* C, int64_t ldc, double* D, int64_t ldd) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i) {
        for (int64_t j = 0; j < n; ++j) {
            dd rr = {0, 0}, ii = {0, 0}, ri = {0, 0}, ir = {0, 0};
            double d = 0.0;
            for (int pass = 0; pass < 2; ++pass) {
                const double* A = pass ? A2 : A1;
                const double* B = pass ? B2 : B1;
                const int64_t lda = pass ? lda2 : lda1, ldb = pass ? ldb2 : ldb1;
                for (int64_t p = 0; p < k; ++p) {
                    double ar = A[2 * (i + p * lda)], ai = A[2 * (i + p * lda) + 1];
                    double br = B[2 * (p + j * ldb)], bi = B[2 * (p + j * ldb) + 1];
                    rr = dd_mac(rr, ar, br);
                    ii = dd_mac(ii, ai, bi);
                    ri = dd_mac(ri, ar, bi);
                    ir = dd_mac(ir, ai, br);
                    d += hypot(ar, ai) * hypot(br, bi);
                }
            }
            dd r = dd_add(rr, dd_neg(ii));
            dd im = dd_add(ri, ir);
            C[2 * (i + j * ldc)] = r.hi + r.lo;
            C[2 * (i + j * ldc) + 1] = im.hi + im.lo;
            D[i + j * ldd] = d;
        }
    }
}

// Pieces shared by the post-processing kernels that form the digit-column sums of the CRT on the tensor cores (post_fp.cu for the
// complex GEMMs, post_herk.cu for the rank-k family): the warp-level MMA wrappers, the packing of four digit-column sums into
// one 64-bit chunk, and the FP64 finish of one part of one element.
#pragma once
#include "post_common.cuh"

namespace gemm2m {

// Words per element in the exchange buffer: 2 parts x NB chunks of 8 bytes, plus a pad that keeps the 16-byte accesses of a
// warp on distinct banks.
__host__ __device__ constexpr int pf_row_words(int nb) { return 4 * nb + 4; }
// D = A B, A: 16 x 32 bytes (row-major fragments), B: 32 x 8 bytes (column-major fragments), D: 16 x 8 int32; unsigned bytes.
__device__ __forceinline__ void mma_u8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "r"(0));
}
// A operand straight from shared memory: 16 (x1) or 32 (x2) rows of 16 bytes, row r = the bytes of K index r for 16
// consecutive elements, loaded transposed.  Lane (g, t) receives, per 16 rows, the bytes of K = 4t .. 4t+3 for element g and
// for element g + 8: the A fragment of the 8-bit MMAs.  Lanes 0..15 (x2: 0..31) supply the row addresses (16-byte aligned).
__device__ __forceinline__ void load_a_k16(uint32_t (&a)[2], uint32_t row_addr) {
    asm volatile("ldmatrix.sync.aligned.m16n16.x1.trans.shared.b8 {%0, %1}, [%2];" : "=r"(a[0]), "=r"(a[1]) : "r"(row_addr) : "memory");
}
__device__ __forceinline__ void load_a_k32(uint32_t (&a)[4], uint32_t row_addr) {
    asm volatile("ldmatrix.sync.aligned.m16n16.x2.trans.shared.b8 {%0, %1, %2, %3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]) : "r"(row_addr) : "memory");
}
// The same with K = 16 (A: 16 x 16, B: 16 x 8): for operands of at most 16 planes.
__device__ __forceinline__ void mma_u8_k16(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm("mma.sync.aligned.m16n8k16.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%7,%7,%7,%7};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(b0), "r"(0));
}
__device__ __forceinline__ void mma_u8_acc(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// hi:lo = b 2^16 + (hi_word 2^32 + a): four digit-column sums s0..s3 packed as a = s0 + 2^8 s1, b = s2 + 2^8 s3 (both below
// 2^31) under the high word of a double, one wide multiply-add.
// (two16 holds 65536 in a register: with the constant in the instruction the compiler splits the product into a shift pair.)
__device__ __forceinline__ unsigned long long pack_chunk(uint32_t a, uint32_t b, uint32_t hi_word, uint32_t two16) {
    unsigned long long r;
    asm("{\n\t.reg .b64 c;\n\tmov.b64 c, {%1, %2};\n\tmad.wide.u32 %0, %3, %4, c;\n\t}" : "=l"(r) : "r"(a), "r"(hi_word), "r"(b), "r"(two16));
    return r;
}

// Lifted X (exact integer, |X| <= M/2) of one part from its NB chunks, returned as an unevaluated sum hi + lo (not
// normalised: lo collects the error terms of the additions, whose own sum is rounded: X = hi + lo up to a few 2^-106 of the
// largest intermediate sum, which exceeds |X| only where chunks cancel, i.e. for entries far below the scale of their row and column).  Chunk k arrives as the bit pattern of the double (1.5 2^52 + V_k) 2^(32k), with
// V_k = s_4k + 2^8 s_(4k+1) + 2^16 s_(4k+2) + 2^24 s_(4k+3) < 2^46.1 the four digit-column sums it covers; off[k] takes the
// conversion offset and the chunk's share of 128 sum_planes W_p off again, exactly, which leaves W_k with
// X' = sum_k W_k 2^(32k) = sum_planes residue_p W_p = X + t M.
// t = rint(X'/M) from the three leading chunks: M >= 2^(32 NB - 64) (its bytes fill more than NB - 2 chunks), so the
// rest is below 2^-17 M; |t| < 2^14, and |X/M| stays away from 1/2 by the scaling rule.  W_k - t Mc_k is exact
// (|t Mc_k| < 2^46 before the weight).  The chunks are then added with error-free transformations, neighbours first (below; two chunks: hi alone is X rounded once, lo = 0).
template <int NB>
__device__ __forceinline__ void crt_finish32(const double (&bits)[NB], const double (&off)[kPostMaxNB], const PostConsts& pc, double* hi, double* lo) {
    double W[NB];
#pragma unroll
    for (int k = 0; k < NB; ++k) W[k] = bits[k] - off[k];
    double lead = W[NB - 1];
#pragma unroll
    for (int k = NB - 2; k >= 0 && k >= NB - 3; --k) lead += W[k];
    const double t = rint(lead * pc.inv_M);
#pragma unroll
    for (int k = 0; k < NB; ++k) W[k] = fma(-t, pc.Mc[k], W[k]);
    if (NB == 2) {               // two exact terms: their floating-point sum is the correctly rounded X already
        *hi = W[1] + W[0];
        *lo = 0.0;
        return;
    }
    // Error-free additions in three operations each (s = a + b, z = s - a, e = b - z): exact whenever a is a whole multiple of
    // ulp(b), whatever the magnitudes.  First loop: a = W[2k+1] is a multiple of 2^(64k+32), |b| = |W[2k]| < 2^(64k+48) has an ulp
    // of at most 2^(64k-4).  Second loop: h, a rounded sum of pairs above k, is a multiple of 2^(64k+64), and |ph[k]| < 2^(64k+81)
    // has an ulp of at most 2^(64k+29).
    double ph[NB / 2], l = 0.0;
#pragma unroll
    for (int k = 0; k < NB / 2; ++k) {
        const double a = W[2 * k + 1], b = W[2 * k];
        const double s = a + b;
        const double z = s - a;
        l += b - z;
        ph[k] = s;
    }
    double h = ph[NB / 2 - 1];
#pragma unroll
    for (int k = NB / 2 - 2; k >= 0; --k) {
        const double s = h + ph[k];
        const double z = s - h;
        l += ph[k] - z;
        h = s;
    }
    *hi = h;
    *lo = l;
}

template <typename T> __device__ __forceinline__ void store_cplx(T* dst, double re, double im);
template <> __device__ __forceinline__ void store_cplx<double>(double* dst, double re, double im) { *reinterpret_cast<double2*>(dst) = make_double2(re, im); }
template <> __device__ __forceinline__ void store_cplx<float>(float* dst, double re, double im) { *reinterpret_cast<float2*>(dst) = make_float2((float)re, (float)im); }

}  // namespace gemm2m

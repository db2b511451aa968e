// Algorithm 1 steps 4 (Eq. 2c), 5, 6, 7: post-processing of the residue planes of the products (complex GEMM, rank-k family,
// real scheme, exact int64 result), plus the small packing and scaling kernels of the rank-k and extended interfaces.
#include "post_common.cuh"

namespace gemm2m {

// =====================================================================================================
// Steps 4 (Eq. 2c), 5, 6, 7: per output element, fold the 2M post-processing into the CRT weights, sum the
// weighted residues exactly in 40-bit digit columns (FP64 FMAs on integers below 2^53), remove the multiple
// of M, and round the lifted integer once to floating point before scaling by 2^(e_i + f_j).
// =====================================================================================================
// Byte e (0..3) of w as a signed integer: one byte permute that copies the byte and replicates its sign bit.
__device__ __forceinline__ int sbyte(uint32_t w, int e) {
    uint32_t r;       // selector nibble = byte index, + 8 to replicate that byte's sign bit (the __byte_perm intrinsic masks that bit off)
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(w), "r"(0u), "r"(0x8880u + 0x1111u * (uint32_t)e));
    return (int)r;
}

__device__ __forceinline__ double int_to_double(int v) {
    // The conversion instruction: one issue slot on a pipe nothing else here uses.  (Building the double from its bit
    // pattern, 2^52 + 2^31 + v minus the constant, took three slots, one of them on the FP64 pipe the FMAs need; measured
    // 7 % slower for the whole kernel.)
    return (double)v;
}

// Lifted X (exact integer, |X| <= (M-1)/2) from the digit-column sums S[c], returned as an unevaluated sum hi + lo with
// |lo| <= ulp(hi)/2.  The weighted sum X' = sum_c S[c] 2^(40c) is X + t M with |t| < 2^12; |X/M| stays below 0.494 by the
// scaling rule, so rounding X'/M (from the two leading sums; the rest is below 2^-60 M) gives t exactly.
template <int NCH>
__device__ __forceinline__ void crt_finish(double (&S)[NCH], const CrtTable& tab, double* hi, double* lo) {
    const double t = rint(NCH > 1 ? fma(S[NCH - 1], tab.q_hi, S[NCH > 1 ? NCH - 2 : 0] * tab.q_lo) : S[0] * tab.q_hi);
#pragma unroll
    for (int c = 0; c < NCH; ++c) S[c] = fma(-t, tab.Mc[c], S[c]);          // exact: |S[c]| + |t| Mc[c] < 2^53 for every modulus count (host test)
    const double two40 = 1099511627776.0, inv40 = 1.0 / 1099511627776.0;
#pragma unroll
    for (int c = 0; c + 1 < NCH; ++c) {                                     // carry into canonical digits [0, 2^40)
        const double carry = floor(S[c] * inv40);
        S[c] = fma(-carry, two40, S[c]);
        S[c + 1] += carry;
    }
    double h = S[NCH - 1], l = 0.0;                                          // top digit keeps the sign
#pragma unroll
    for (int c = NCH - 2; c >= 0; --c) {
        h *= two40;
        l *= two40;
        const double s = h + S[c];                                           // TwoSum
        const double bb = s - h;
        const double err = (h - (s - bb)) + (S[c] - bb);
        h = s;
        l += err;
    }
    *hi = h;
    *lo = l;
}

constexpr int kPostThreads = 128;
constexpr int kPostSpan = kPostThreads * 4;   // consecutive row indices i handled by one block

// Real Ozaki-II scheme (Section 3.1): cp: [nmod][n][ldp] int8, one plane per modulus; X = sum_j c_j G_j (mod M) with
// G_j = sym(q_j)(M/m_j) in tab.gr; real double output.  Same staging and finish as post_fp_kernel.
template <int NCH>
__global__ void __launch_bounds__(kPostThreads) post_real_kernel(const int8_t* __restrict__ cp, int64_t ldp, int64_t m, int64_t n,
                                                                 const int32_t* __restrict__ eA, const int32_t* __restrict__ eB,
                                                                 const __grid_constant__ CrtTable tab, double* __restrict__ C, int64_t ldc) {
    __shared__ __align__(16) uint32_t stage[kMaxMod][kPostThreads];
    const int64_t ib = (int64_t)blockIdx.x * kPostSpan;
    const int64_t j = blockIdx.y;
    const int nmod = tab.nmod;
    const int64_t plane = n * ldp;
    const int8_t* src = cp + j * ldp + ib;
    const int vec_per_plane = (int)min((int64_t)(kPostSpan / 16), (ldp - ib) / 16);
    for (int idx = threadIdx.x; idx < nmod * (kPostSpan / 16); idx += kPostThreads) {
        const int p = idx / (kPostSpan / 16), v = idx - p * (kPostSpan / 16);
        if (v < vec_per_plane) cp_async16(&stage[p][4 * v], src + (int64_t)p * plane + 16 * v);
    }
    cp_async_wait_all();
    __syncthreads();
    const int64_t i0 = ib + 4 * threadIdx.x;
    if (i0 >= m) return;
    double S[4][NCH];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
#pragma unroll
        for (int c = 0; c < NCH; ++c) S[e][c] = 0.0;
    }
#pragma unroll 2
    for (int jm = 0; jm < nmod; ++jm) {
        const uint32_t w = stage[jm][threadIdx.x];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const double v = int_to_double(sbyte(w, e));
#pragma unroll
            for (int c = 0; c < NCH; ++c) S[e][c] = fma(v, tab.gr[jm][c], S[e][c]);
        }
    }
    const int fb = __ldg(eB + j);
    for (int e = 0; e < 4; ++e) {
        if (i0 + e < m) {
            const int ea = __ldg(eA + i0 + e);
            double out;
            if (ea == kExpNonFinite || fb == kExpNonFinite) {
                out = __longlong_as_double(0x7FF8000000000000ll);
            } else {
                double h, l;
                crt_finish<NCH>(S[e], tab, &h, &l);
                out = scale_pow2(h + l, ea + fb);
            }
            C[i0 + e + j * ldc] = out;
        }
    }
}

cudaError_t launch_post_real(const int8_t* cp, int64_t ldp, int64_t m, int64_t n, int64_t j_begin, int64_t j_end, const int32_t* eA,
                             const int32_t* eB, const CrtTable& tab, double* C, int64_t ldc, cudaStream_t st, int* launches) {
    if (m <= 0 || j_end <= j_begin) return cudaSuccess;
    for (int64_t j0 = j_begin; j0 < j_end; j0 += 65535) {
        const int64_t nj = (j_end - j0 < 65535) ? j_end - j0 : 65535;
        dim3 grid((unsigned)((m + kPostSpan - 1) / kPostSpan), (unsigned)nj);
        const int8_t* src = cp + j0 * ldp;
        double* dst = C + j0 * ldc;
        switch (tab.nchunks) {
            case 1: post_real_kernel<1><<<grid, kPostThreads, 0, st>>>(src, ldp, m, n, eA, eB + j0, tab, dst, ldc); break;
            case 2: post_real_kernel<2><<<grid, kPostThreads, 0, st>>>(src, ldp, m, n, eA, eB + j0, tab, dst, ldc); break;
            case 3: post_real_kernel<3><<<grid, kPostThreads, 0, st>>>(src, ldp, m, n, eA, eB + j0, tab, dst, ldc); break;
            default: post_real_kernel<4><<<grid, kPostThreads, 0, st>>>(src, ldp, m, n, eA, eB + j0, tab, dst, ldc); break;
        }
        ++*launches;
    }
    return cudaGetLastError();
}

// C = beta C (C = 0 for beta = 0, without reading C): the alpha = 0 case of the extended interface.
template <typename T>
__global__ void __launch_bounds__(256) scale_c_kernel(T* __restrict__ C, int64_t m, int64_t n, int64_t ldc, double br, double bi) {
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x, j = blockIdx.y;
    if (i >= m) return;
    T* c = C + 2 * (i + j * ldc);
    double yr = 0.0, yi = 0.0;
    if (br != 0.0 || bi != 0.0) {
        const double cr = (double)c[0], ci = (double)c[1];
        yr = fma(br, cr, -bi * ci);
        yi = fma(br, ci, bi * cr);
    }
    c[0] = (T)yr;
    c[1] = (T)yi;
}

template <typename T>
cudaError_t launch_scale_c(T* C, int64_t m, int64_t n, int64_t ldc, const double* beta, cudaStream_t st, int* launches) {
    if (m <= 0 || n <= 0) return cudaSuccess;
    const double br = beta ? beta[0] : 0.0, bi = beta ? beta[1] : 0.0;
    for (int64_t j0 = 0; j0 < n; j0 += 65535) {
        const int64_t nj = (n - j0 < 65535) ? n - j0 : 65535;
        dim3 grid((unsigned)((m + 255) / 256), (unsigned)nj);
        scale_c_kernel<T><<<grid, 256, 0, st>>>(C + 2 * j0 * ldc, m, nj, ldc, br, bi);
        ++*launches;
    }
    return cudaGetLastError();
}
template cudaError_t launch_scale_c<double>(double*, int64_t, int64_t, int64_t, const double*, cudaStream_t, int*);
template cudaError_t launch_scale_c<float>(float*, int64_t, int64_t, int64_t, const double*, cudaStream_t, int*);

__global__ void __launch_bounds__(256) pack_real_pair_kernel(const double* __restrict__ X, int64_t ld, int64_t n, int64_t k, int64_t k2,
                                                             double* __restrict__ Z) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t p = blockIdx.y;
    if (i >= n) return;
    const double re = __ldg(X + i + p * ld);
    const double im = (p + k2 < k) ? __ldg(X + i + (p + k2) * ld) : 0.0;
    *reinterpret_cast<double2*>(Z + 2 * (i + p * n)) = make_double2(re, im);
}

cudaError_t launch_pack_real_pair(const double* X, int64_t ld, int64_t n, int64_t k, double* Z, cudaStream_t st, int* launches) {
    const int64_t k2 = (k + 1) / 2;
    if (n <= 0 || k2 <= 0) return cudaSuccess;
    for (int64_t p0 = 0; p0 < k2; p0 += 65535) {      // grid.y limit
        const int64_t np = (k2 - p0 < 65535) ? k2 - p0 : 65535;
        dim3 grid((unsigned)((n + 255) / 256), (unsigned)np);
        pack_real_pair_kernel<<<grid, 256, 0, st>>>(X + p0 * ld, ld, n, k - p0, k2, Z + 2 * p0 * n);
        ++*launches;
    }
    return cudaGetLastError();
}

// Exact integer variant for gemm2m_gaussian_int: X = sum_j sym(v_j g_j mod m_j) (M/m_j) mod M in int64 (M < 2^62).
__global__ void __launch_bounds__(256) post_int_kernel(const int8_t* __restrict__ cpm, int64_t ldp, int64_t m, int64_t n,
                                                       const __grid_constant__ CrtTableInt tab, int64_t* __restrict__ Cr,
                                                       int64_t* __restrict__ Ci, int64_t ldc) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t j = blockIdx.y;
    if (i >= m) return;
    const int nmod = tab.nmod;
    const int64_t plane = n * ldp;
    const int8_t* src = cpm + j * ldp + i;
    long long xr = 0, xi = 0;
    const long long M = tab.M;
    for (int jm = 0; jm < nmod; ++jm) {
        const int cp = src[(int64_t)jm * plane], cm = src[(int64_t)(nmod + jm) * plane];
        const int mj = tab.m[jm], half = (mj - 1) / 2;
        int ur = ((cm + cp) * tab.gr[jm]) % mj;       // Eq. (2c) and the CRT factor q_j, folded
        int ui = ((cm - cp) * tab.gi[jm]) % mj;
        if (ur > half) ur -= mj; else if (ur < -half) ur += mj;
        if (ui > half) ui -= mj; else if (ui < -half) ui += mj;
        xr = (xr + (long long)ur * tab.W[jm]) % M;    // |term| < 2^62, |xr| < M < 2^62: no overflow
        xi = (xi + (long long)ui * tab.W[jm]) % M;
    }
    const long long h = (M - 1) / 2;                  // lift to [-(M-1)/2, (M-1)/2]
    if (xr > h) xr -= M; else if (xr < -h) xr += M;
    if (xi > h) xi -= M; else if (xi < -h) xi += M;
    Cr[i + j * ldc] = xr;
    Ci[i + j * ldc] = xi;
}

cudaError_t launch_post_int(const int8_t* cpm, int64_t ldp, int64_t m, int64_t n, const CrtTableInt& tab, int64_t* Cr, int64_t* Ci,
                            int64_t ldc, cudaStream_t st, int* launches) {
    if (m <= 0 || n <= 0) return cudaSuccess;
    for (int64_t j0 = 0; j0 < n; j0 += 65535) {
        const int64_t nj = (n - j0 < 65535) ? n - j0 : 65535;
        dim3 grid((unsigned)((m + 255) / 256), (unsigned)nj);
        post_int_kernel<<<grid, 256, 0, st>>>(cpm + j0 * ldp, ldp, m, n, tab, Cr + j0 * ldc, Ci + j0 * ldc, ldc);
        ++*launches;
    }
    return cudaGetLastError();
}



}  // namespace gemm2m

// Pre- and post-processing kernels of 2M Ozaki-II (Algorithm 1 steps 2, 3, 4 (Eq. 2a, 2c), 5, 6, 7).
// All of them are streaming kernels bounded by HBM bandwidth / plain ALU throughput.
#include "common.cuh"

namespace gemm2m {

// =====================================================================================================
// Step 2: exponent scan.  For every row (or column) the largest magnitude bit pattern of any real or
// imaginary part; IEEE bit patterns of non-negative numbers are ordered like the numbers themselves.
// =====================================================================================================
template <typename T> struct FpBits;
template <> struct FpBits<double> {
    using U = unsigned long long;
    static constexpr int kMantBits = 52, kExpMax = 2047, kBias = 1023;
    __device__ static U mag(double v) { return (U)__double_as_longlong(v) & 0x7FFFFFFFFFFFFFFFull; }
};
template <> struct FpBits<float> {
    using U = unsigned long long;
    static constexpr int kMantBits = 23, kExpMax = 255, kBias = 127;
    __device__ static U mag(float v) { return (U)(__float_as_uint(v) & 0x7FFFFFFFu); }
};

template <typename T> struct Cplx { T re, im; };
template <typename T> __device__ __forceinline__ Cplx<T> load_cplx(const T* p);
template <> __device__ __forceinline__ Cplx<double> load_cplx<double>(const double* p) {
    const double2 v = __ldg(reinterpret_cast<const double2*>(p));
    return {v.x, v.y};
}
template <> __device__ __forceinline__ Cplx<float> load_cplx<float>(const float* p) {
    const float2 v = __ldg(reinterpret_cast<const float2*>(p));
    return {v.x, v.y};
}

static int cached_sm_count() {
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            sms = 148;
    }
    return sms;
}

constexpr int kScanThreads = 256;
constexpr int kScanRowsSpan = 64;     // columns handled by one block of scan_rows
constexpr int kScanColsSpan = 2048;   // rows handled by one warp of scan_cols

// One thread per row, a span of columns per block: consecutive threads read consecutive rows (coalesced).
template <typename T>
__global__ void __launch_bounds__(kScanThreads) scan_rows_kernel(const T* __restrict__ X, int64_t rows, int64_t cols, int64_t ld, int64_t span,
                                                                 unsigned long long* __restrict__ absmax) {
    const int64_t r = (int64_t)blockIdx.x * kScanThreads + threadIdx.x;
    if (r >= rows) return;
    const int64_t c0 = (int64_t)blockIdx.y * span;
    const int64_t c1 = min(cols, c0 + span);
    unsigned long long mx = 0;
    const T* p = X + 2 * (r + c0 * ld);
#pragma unroll 8
    for (int64_t c = c0; c < c1; ++c, p += 2 * ld) {
        const Cplx<T> v = load_cplx<T>(p);
        mx = max(mx, max(FpBits<T>::mag(v.re), FpBits<T>::mag(v.im)));
    }
    if (mx) atomicMax(absmax + r, mx);
}

// One warp per (column, span of rows): lanes read consecutive elements of the column.
template <typename T>
__global__ void __launch_bounds__(kScanThreads) scan_cols_kernel(const T* __restrict__ X, int64_t rows, int64_t cols, int64_t ld, int64_t span,
                                                                 unsigned long long* __restrict__ absmax) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c = (int64_t)blockIdx.x * (kScanThreads / 32) + warp;
    if (c >= cols) return;
    const int64_t r0 = (int64_t)blockIdx.y * span;
    const int64_t r1 = min(rows, r0 + span);
    unsigned long long mx = 0;
    const T* base = X + 2 * (c * ld);
#pragma unroll 4
    for (int64_t r = r0 + lane; r < r1; r += 32) {
        const Cplx<T> v = load_cplx<T>(base + 2 * r);
        mx = max(mx, max(FpBits<T>::mag(v.re), FpBits<T>::mag(v.im)));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    if (lane == 0 && mx) atomicMax(absmax + c, mx);
}

// e = floor(log2 mu) + 1 + c_k - P for the largest magnitude mu; 0 for an all-zero row; sentinel for Inf/NaN.
template <typename T>
__global__ void exponents_kernel(const unsigned long long* __restrict__ absmax, int64_t count, int P, int ck, int32_t* __restrict__ e) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const unsigned long long b = absmax[i];
    int out;
    if (b == 0) {
        out = 0;
    } else {
        const int E = (int)(b >> FpBits<T>::kMantBits);
        if (E == FpBits<T>::kExpMax) {
            out = kExpNonFinite;
        } else {
            const int x = E ? E - FpBits<T>::kBias : (63 - __clzll((long long)b)) - (FpBits<T>::kBias - 1 + FpBits<T>::kMantBits);
            out = x + 1 + ck - P;
        }
    }
    e[i] = out;
}

// ---- real matrices (real Ozaki-II scheme, Section 3.1): the same scans over scalar elements ----------------
template <typename T>
__global__ void __launch_bounds__(kScanThreads) scan_rows_real_kernel(const T* __restrict__ X, int64_t rows, int64_t cols, int64_t ld, int64_t span,
                                                                      unsigned long long* __restrict__ absmax) {
    const int64_t r = (int64_t)blockIdx.x * kScanThreads + threadIdx.x;
    if (r >= rows) return;
    const int64_t c0 = (int64_t)blockIdx.y * span;
    const int64_t c1 = min(cols, c0 + span);
    unsigned long long mx = 0;
    const T* p = X + (r + c0 * ld);
#pragma unroll 8
    for (int64_t c = c0; c < c1; ++c, p += ld) mx = max(mx, FpBits<T>::mag(__ldg(p)));
    if (mx) atomicMax(absmax + r, mx);
}

template <typename T>
__global__ void __launch_bounds__(kScanThreads) scan_cols_real_kernel(const T* __restrict__ X, int64_t rows, int64_t cols, int64_t ld, int64_t span,
                                                                      unsigned long long* __restrict__ absmax) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c = (int64_t)blockIdx.x * (kScanThreads / 32) + warp;
    if (c >= cols) return;
    const int64_t r0 = (int64_t)blockIdx.y * span;
    const int64_t r1 = min(rows, r0 + span);
    unsigned long long mx = 0;
    const T* base = X + c * ld;
#pragma unroll 4
    for (int64_t r = r0 + lane; r < r1; r += 32) mx = max(mx, FpBits<T>::mag(__ldg(base + r)));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    if (lane == 0 && mx) atomicMax(absmax + c, mx);
}

template <typename T>
cudaError_t launch_scan_real(const T* X, int64_t rows, int64_t cols, int64_t ld, bool per_row, uint64_t* absmax, cudaStream_t st, int* launches) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    if (per_row) {
        int64_t span = kScanRowsSpan;
        while ((cols + span - 1) / span > 65535) span *= 2;
        dim3 grid((unsigned)((rows + kScanThreads - 1) / kScanThreads), (unsigned)((cols + span - 1) / span));
        scan_rows_real_kernel<T><<<grid, kScanThreads, 0, st>>>(X, rows, cols, ld, span, (unsigned long long*)absmax);
    } else {
        int64_t span = 2 * kScanColsSpan;
        while ((rows + span - 1) / span > 65535) span *= 2;
        dim3 grid((unsigned)((cols + kScanThreads / 32 - 1) / (kScanThreads / 32)), (unsigned)((rows + span - 1) / span));
        scan_cols_real_kernel<T><<<grid, kScanThreads, 0, st>>>(X, rows, cols, ld, span, (unsigned long long*)absmax);
    }
    ++*launches;
    return cudaGetLastError();
}
template cudaError_t launch_scan_real<double>(const double*, int64_t, int64_t, int64_t, bool, uint64_t*, cudaStream_t, int*);

// ---- 2-norm scaling rule: second pass over the operand --------------------------------------------------
// floor(log2) of the finite non-zero magnitude with bit pattern b.
template <typename T>
__device__ __forceinline__ int floor_log2_bits(unsigned long long b) {
    const int E = (int)(b >> FpBits<T>::kMantBits);
    return E ? E - FpBits<T>::kBias : (63 - __clzll((long long)b)) - (FpBits<T>::kBias - 1 + FpBits<T>::kMantBits);
}
// u = ceil(|v| 2^(20 - (x+1))) for a part with bit pattern b, |v| < 2^(x+1): an integer in [0, 2^20].
template <typename T>
__device__ __forceinline__ unsigned long long fixed_mag_up(unsigned long long b, int x) {
    if (b == 0) return 0;
    const int E = (int)(b >> FpBits<T>::kMantBits);
    unsigned long long mant = b & ((1ull << FpBits<T>::kMantBits) - 1);
    if (E) mant |= (1ull << FpBits<T>::kMantBits);
    // |v| = mant 2^(max(E,1) - bias - mantbits), so u = ceil(mant 2^-r) with r > 0 because max(E,1) - bias <= x
    const int r = -(max(E, 1) - (FpBits<T>::kBias + FpBits<T>::kMantBits) + 19 - x);
    if (r >= 64) return 1;
    return (mant + ((1ull << r) - 1)) >> r;
}

template <typename T>
__global__ void __launch_bounds__(kScanThreads) sumsq_rows_kernel(const T* __restrict__ X, int64_t rows, int64_t cols, int64_t ld, int64_t span,
                                                                  const unsigned long long* __restrict__ absmax,
                                                                  unsigned long long* __restrict__ qsum) {
    const int64_t r = (int64_t)blockIdx.x * kScanThreads + threadIdx.x;
    if (r >= rows) return;
    const unsigned long long b = absmax[r];
    if (b == 0 || (int)(b >> FpBits<T>::kMantBits) == FpBits<T>::kExpMax) return;
    const int x = floor_log2_bits<T>(b);
    const int64_t c0 = (int64_t)blockIdx.y * span;
    const int64_t c1 = min(cols, c0 + span);
    unsigned long long q = 0;
    const T* p = X + 2 * (r + c0 * ld);
#pragma unroll 8
    for (int64_t c = c0; c < c1; ++c, p += 2 * ld) {
        const Cplx<T> v = load_cplx<T>(p);
        const unsigned long long ur = fixed_mag_up<T>(FpBits<T>::mag(v.re), x), ui = fixed_mag_up<T>(FpBits<T>::mag(v.im), x);
        q += ur * ur + ui * ui;
    }
    if (q) atomicAdd(qsum + r, q);
}

template <typename T>
__global__ void __launch_bounds__(kScanThreads) sumsq_cols_kernel(const T* __restrict__ X, int64_t rows, int64_t cols, int64_t ld, int64_t span,
                                                                  const unsigned long long* __restrict__ absmax,
                                                                  unsigned long long* __restrict__ qsum) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c = (int64_t)blockIdx.x * (kScanThreads / 32) + warp;
    if (c >= cols) return;
    const unsigned long long b = absmax[c];
    if (b == 0 || (int)(b >> FpBits<T>::kMantBits) == FpBits<T>::kExpMax) return;
    const int x = floor_log2_bits<T>(b);
    const int64_t r0 = (int64_t)blockIdx.y * span;
    const int64_t r1 = min(rows, r0 + span);
    unsigned long long q = 0;
    const T* base = X + 2 * (c * ld);
#pragma unroll 4
    for (int64_t r = r0 + lane; r < r1; r += 32) {
        const Cplx<T> v = load_cplx<T>(base + 2 * r);
        const unsigned long long ur = fixed_mag_up<T>(FpBits<T>::mag(v.re), x), ui = fixed_mag_up<T>(FpBits<T>::mag(v.im), x);
        q += ur * ur + ui * ui;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) q += __shfl_xor_sync(0xffffffffu, q, off);
    if (lane == 0 && q) atomicAdd(qsum + c, q);
}

// e = x + 1 - P + (t - 20), t the smallest integer with 4^t >= Q (Q = sum of the squared fixed-point magnitudes).
template <typename T>
__global__ void exponents_2norm_kernel(const unsigned long long* __restrict__ absmax, const unsigned long long* __restrict__ qsum, int64_t count,
                                       int P, int32_t* __restrict__ e) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const unsigned long long b = absmax[i];
    int out = 0;
    if (b != 0) {
        if ((int)(b >> FpBits<T>::kMantBits) == FpBits<T>::kExpMax) {
            out = kExpNonFinite;
        } else {
            const unsigned long long Q = qsum[i];
            const int L = Q > 1 ? 64 - __clzll((long long)(Q - 1)) : 0;      // ceil(log2 Q)
            out = floor_log2_bits<T>(b) + 1 - P + ((L + 1) >> 1) - 20;
        }
    }
    e[i] = out;
}

template <typename T>
cudaError_t launch_exponents_2norm(const T* X, int64_t rows, int64_t cols, int64_t ld, bool per_row, const uint64_t* absmax, uint64_t* qsum,
                                   int P, int32_t* e, cudaStream_t st, int* launches) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    const unsigned long long* am = (const unsigned long long*)absmax;
    unsigned long long* qs = (unsigned long long*)qsum;
    if (per_row) {
        int64_t span = kScanRowsSpan;
        while ((cols + span - 1) / span > 65535) span *= 2;
        dim3 grid((unsigned)((rows + kScanThreads - 1) / kScanThreads), (unsigned)((cols + span - 1) / span));
        sumsq_rows_kernel<T><<<grid, kScanThreads, 0, st>>>(X, rows, cols, ld, span, am, qs);
    } else {
        int64_t span = kScanColsSpan;
        while ((rows + span - 1) / span > 65535) span *= 2;
        dim3 grid((unsigned)((cols + kScanThreads / 32 - 1) / (kScanThreads / 32)), (unsigned)((rows + span - 1) / span));
        sumsq_cols_kernel<T><<<grid, kScanThreads, 0, st>>>(X, rows, cols, ld, span, am, qs);
    }
    ++*launches;
    const int64_t count = per_row ? rows : cols;
    exponents_2norm_kernel<T><<<(unsigned)((count + 255) / 256), 256, 0, st>>>(am, qs, count, P, e);
    ++*launches;
    return cudaGetLastError();
}
template cudaError_t launch_exponents_2norm<double>(const double*, int64_t, int64_t, int64_t, bool, const uint64_t*, uint64_t*, int, int32_t*, cudaStream_t, int*);
template cudaError_t launch_exponents_2norm<float>(const float*, int64_t, int64_t, int64_t, bool, const uint64_t*, uint64_t*, int, int32_t*, cudaStream_t, int*);

template <typename T>
cudaError_t launch_scan_rows(const T* X, int64_t rows, int64_t cols, int64_t ld, uint64_t* absmax, cudaStream_t st, int* launches) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    int64_t span = kScanRowsSpan;
    const int64_t row_blocks = (rows + kScanThreads - 1) / kScanThreads;
    while (span > 8 && row_blocks * ((cols + span - 1) / span) < 4 * cached_sm_count()) span /= 2;   // small matrices: enough blocks to fill the GPU
    while ((cols + span - 1) / span > 65535) span *= 2;        // grid.y limit
    dim3 grid((unsigned)row_blocks, (unsigned)((cols + span - 1) / span));
    scan_rows_kernel<T><<<grid, kScanThreads, 0, st>>>(X, rows, cols, ld, span, (unsigned long long*)absmax);
    ++*launches;
    return cudaGetLastError();
}
template <typename T>
cudaError_t launch_scan_cols(const T* X, int64_t rows, int64_t cols, int64_t ld, uint64_t* absmax, cudaStream_t st, int* launches) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    int64_t span = kScanColsSpan;
    const int64_t col_blocks = (cols + kScanThreads / 32 - 1) / (kScanThreads / 32);
    while (span > 256 && col_blocks * ((rows + span - 1) / span) < 4 * cached_sm_count()) span /= 2;
    while ((rows + span - 1) / span > 65535) span *= 2;        // grid.y limit
    dim3 grid((unsigned)col_blocks, (unsigned)((rows + span - 1) / span));
    scan_cols_kernel<T><<<grid, kScanThreads, 0, st>>>(X, rows, cols, ld, span, (unsigned long long*)absmax);
    ++*launches;
    return cudaGetLastError();
}
template <typename T>
cudaError_t launch_exponents(const uint64_t* absmax, int64_t count, int P, int ck, int32_t* e, cudaStream_t st, int* launches) {
    if (count <= 0) return cudaSuccess;
    exponents_kernel<T><<<(unsigned)((count + 255) / 256), 256, 0, st>>>((const unsigned long long*)absmax, count, P, ck, e);
    ++*launches;
    return cudaGetLastError();
}

// =====================================================================================================
// Steps 3 + 4 (Eq. 2a): quantise by truncation and emit the symmetric int8 residues A+ / A- for every
// modulus, K contiguous.  Tiles of operand rows x 128 k are staged in shared memory (coalesced global
// reads in either orientation), then each thread owns a run of consecutive k of one row and writes
// vectors into every plane.
// =====================================================================================================
struct QPair { long long re, im; };   // quantised parts, two's complement

// trunc(v 2^-e) for a finite v given by its bit pattern; the scaling rule guarantees |result| < 2^62 in the narrow mode.
template <typename T>
__device__ __forceinline__ long long quantise_part(T v, int e) {
    using F = FpBits<T>;
    const unsigned long long mag = F::mag(v);
    const int E = (int)(mag >> F::kMantBits);
    unsigned long long mant = mag & ((1ull << F::kMantBits) - 1);
    if (E) mant |= (1ull << F::kMantBits);
    // v = mant 2^(max(E,1) - bias - mantbits)
    const int sh = max(E, 1) - (F::kBias + F::kMantBits) - e;
    const bool neg = (sizeof(T) == 8) ? (__double_as_longlong((double)v) < 0) : (__float_as_int((float)v) < 0);
    unsigned long long q;
    if (sh >= 0) q = mant << min(sh, 63);
    else q = (-sh > 63) ? 0ull : (mant >> (-sh));
    return neg ? -(long long)q : (long long)q;
}

// Wide mode: |result| < 2^92 (19 or more moduli; 2^76 without the hybrid's 3M moduli); returned as the low 32 bits and the
// signed upper 64 bits of the 96-bit two's complement value.
template <typename T>
__device__ __forceinline__ void quantise_part_wide(T v, int e, uint32_t* lo, long long* upper) {
    using F = FpBits<T>;
    const unsigned long long mag = F::mag(v);
    const int E = (int)(mag >> F::kMantBits);
    unsigned long long mant = mag & ((1ull << F::kMantBits) - 1);
    if (E) mant |= (1ull << F::kMantBits);
    const int sh = max(E, 1) - (F::kBias + F::kMantBits) - e;
    const bool neg = (sizeof(T) == 8) ? (__double_as_longlong((double)v) < 0) : (__float_as_int((float)v) < 0);
    unsigned __int128 q;
    if (sh >= 0) q = (unsigned __int128)mant << min(sh, 74);   // a legitimate shift stays below 92 - 23; the clamp only keeps the shift defined
    else q = (-sh > 63) ? 0 : (mant >> (-sh));
    const __int128 sq = neg ? -(__int128)q : (__int128)q;
    *lo = (uint32_t)(unsigned __int128)sq;
    *upper = (long long)(sq >> 32);
}

__device__ __forceinline__ int dp4a_us(uint32_t a_unsigned, uint32_t b_signed, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a_unsigned), "r"(b_signed), "r"(c));
    return d;
}
__device__ __forceinline__ int dp4a_ss(uint32_t a_signed, uint32_t b_signed, int c) {
    int d;
    asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a_signed), "r"(b_signed), "r"(c));
    return d;
}

// Symmetric residues of the pair of sums x+ = Rv + Iv and x- = Rv - Iv, returned in the low bytes of bp / bm (two's
// complement).  The caller starts the dp4a chain at the bit pattern of the float Y0 = a multiple of 256 m in [2^23, 2^24),
// so the integers yp = bits(Y0) + x+ and ym = bits(Y0) + x- are the bit patterns of the floats Y0 + x.  One FMA with the
// constant cq = 1.5 2^23 - Y0/m gives t = 1.5 2^23 + rint(x/m) exactly (the table builder proves that the error of inv_m
// stays below the distance of x/m from a rounding boundary), and bits(y) - bits(t) m has the low byte of x - rint(x/m) m
// because the bit patterns of Y0 and of 1.5 2^23 are multiples of 256.  Per residue: one FP32 FMA, one integer multiply-add.
__device__ __forceinline__ void sym_reduce_pm(int yp, int ym, int neg_m, float inv_m, float cq, uint32_t* bp, uint32_t* bm) {
    const int tp = __float_as_int(fmaf(__int_as_float(yp), inv_m, cq));
    const int tm = __float_as_int(fmaf(__int_as_float(ym), inv_m, cq));
    *bp = (uint32_t)(tp * neg_m + yp);
    *bm = (uint32_t)(tm * neg_m + ym);
}

struct Digits { uint32_t lo, hi; };   // 4 unsigned low bytes; 4 balanced (signed) high digits
__device__ __forceinline__ Digits split_digits(long long x) {
    Digits d;
    d.lo = (uint32_t)(unsigned long long)x;
    const uint32_t hi = (uint32_t)((unsigned long long)x >> 32);
    d.hi = (hi + 0x80808080u) ^ 0x80808080u;   // hi = sum (byte_b - 128) 256^b  after adding 128 to every byte
    return d;
}
// The same for a 96-bit value given as low word and signed upper 64 bits: 8 balanced digits above the low word.
__device__ __forceinline__ Digits split_digits_wide(uint32_t lo, long long upper, uint32_t* top) {
    const unsigned long long rec = ((unsigned long long)upper + 0x8080808080808080ull) ^ 0x8080808080808080ull;
    Digits d;
    d.lo = lo;
    d.hi = (uint32_t)rec;
    *top = (uint32_t)(rec >> 32);
    return d;
}

// One symmetric residue from y = bits(Y0) + x (see sym_reduce_pm).
__device__ __forceinline__ uint32_t sym_reduce_one(int y, int neg_m, float inv_m, float cq) {
    const int t = __float_as_int(fmaf(__int_as_float(y), inv_m, cq));
    return (uint32_t)(t * neg_m + y);
}

__device__ __forceinline__ uint32_t pack4(const uint32_t (&b)[4]) {   // low bytes of four words -> one word
    return __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
}

template <int NE>
__device__ __forceinline__ void store_run(int8_t* dst, const uint32_t (&w)[NE / 4]) {
    if (NE == 16) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2 % (NE / 4)], w[3 % (NE / 4)]);
    else *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
}

// One 2M modulus (index j) of emit_run: X+ into plane j, X- into plane n2 + j.
template <int NE, bool WIDE>
__device__ __forceinline__ void emit_2m(int j, int n2, const Digits (&dr)[NE], const Digits (&di)[NE], const uint32_t* tr, const uint32_t* ti,
                                        const ResidueTable& tab, int8_t* dst, int64_t plane_stride) {
    const int neg_m = -tab.m[j], y0 = tab.magic[j];
    const float inv_m = tab.inv_m[j], cq = tab.cq[j];
    const uint32_t wl = tab.w_lo[j], wh = tab.w_hi[j], sl = tab.ws_lo[j], sh = tab.ws_hi[j];
    const uint32_t wt = WIDE ? tab.w_top[j] : 0u, st = WIDE ? tab.ws_top[j] : 0u;
    uint32_t pw[NE / 4], mw[NE / 4];
#pragma unroll
    for (int w = 0; w < NE / 4; ++w) {
        uint32_t bp[4], bm[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int i = 4 * w + b;
            int Ry = dp4a_ss(dr[i].hi, wh, dp4a_us(dr[i].lo, wl, y0));  // A_r mod m (unreduced) on top of the bits of Y0
            if (WIDE) Ry = dp4a_ss(tr[i], wt, Ry);                      // digits 8..11 of the 96-bit value
            // The imaginary part's weights continue the same chain: no separate addition for the "+" sum of Eq. (2a),
            // and the "-" sum is 2 Ry - yp, a three-input integer add that does not compete with the dp4a's for their pipe.
            int yp = dp4a_ss(di[i].hi, sh, dp4a_us(di[i].lo, sl, Ry));
            if (WIDE) yp = dp4a_ss(ti[i], st, yp);
            const int ym = (int)(2u * (uint32_t)Ry - (uint32_t)yp);     // the doubled bit pattern wraps, the difference does not
            sym_reduce_pm(yp, ym, neg_m, inv_m, cq, &bp[b], &bm[b]);
        }
        pw[w] = pack4(bp);
        mw[w] = pack4(bm);
    }
    store_run<NE>(dst + (int64_t)j * plane_stride, pw);
    store_run<NE>(dst + (int64_t)(n2 + j) * plane_stride, mw);
}

// Residues of NE consecutive elements of one operand row for every modulus, written as NE-byte vectors into the planes of
// that modulus: X+ and X- (Eq. 2a) for the 2M moduli, then X_r, X_i and X_r + X_i (Eq. 1 after the reduction) for the 3M
// moduli of the hybrid.  dst points at plane 0, this row, first k of the run; tr / ti (wide mode) hold the four top digits
// of each part.  NMOD > 0: exactly NMOD moduli, all of them 2M moduli, known at compile time: the loop is unrolled and the
// per-modulus constants become constant-bank operands instead of loads.
template <int NE, bool WIDE, int NMOD>
__device__ __forceinline__ void emit_run(const Digits (&dr)[NE], const Digits (&di)[NE], const uint32_t* tr, const uint32_t* ti,
                                         const ResidueTable& tab, int8_t* dst, int64_t plane_stride) {
    static_assert(NE == 8 || NE == 16, "runs of 8 or 16 elements");
    if constexpr (NMOD > 0) {
#pragma unroll
        for (int j = 0; j < NMOD; ++j) emit_2m<NE, WIDE>(j, NMOD, dr, di, tr, ti, tab, dst, plane_stride);
        return;
    }
    const int nmod = tab.nmod, n2 = tab.n2;
#pragma unroll 1
    for (int j = 0; j < n2; ++j) emit_2m<NE, WIDE>(j, n2, dr, di, tr, ti, tab, dst, plane_stride);
    const int n3 = nmod - n2;
    int8_t* dst3 = dst + (int64_t)(2 * n2) * plane_stride;
#pragma unroll 1
    for (int j3 = 0; j3 < n3; ++j3) {
        const int j = n2 + j3;
        const int neg_m = -tab.m[j], y0 = tab.magic[j];
        const float inv_m = tab.inv_m[j], cq = tab.cq[j];
        const uint32_t wl = tab.w_lo[j], wh = tab.w_hi[j], wt = WIDE ? tab.w_top[j] : 0u;
        uint32_t rw[NE / 4], iw[NE / 4], sw[NE / 4];
#pragma unroll
        for (int w = 0; w < NE / 4; ++w) {
            uint32_t br[4], bi[4], bs[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int i = 4 * w + b;
                int Ry = dp4a_ss(dr[i].hi, wh, dp4a_us(dr[i].lo, wl, y0));  // A_r mod m (unreduced) on top of the bits of Y0
                if (WIDE) Ry = dp4a_ss(tr[i], wt, Ry);
                int ys = dp4a_ss(di[i].hi, wh, dp4a_us(di[i].lo, wl, Ry));  // A_r + A_i: the same weights for both parts
                if (WIDE) ys = dp4a_ss(ti[i], wt, ys);
                const int Iy = ys - Ry + y0;                                // A_i alone
                br[b] = sym_reduce_one(Ry, neg_m, inv_m, cq);
                bi[b] = sym_reduce_one(Iy, neg_m, inv_m, cq);
                bs[b] = sym_reduce_one(ys, neg_m, inv_m, cq);
            }
            rw[w] = pack4(br);
            iw[w] = pack4(bi);
            sw[w] = pack4(bs);
        }
        store_run<NE>(dst3 + (int64_t)j3 * plane_stride, rw);
        store_run<NE>(dst3 + (int64_t)(n3 + j3) * plane_stride, iw);
        store_run<NE>(dst3 + (int64_t)(2 * n3 + j3) * plane_stride, sw);
    }
}

// ---- floating-point inputs: persistent blocks, raw elements copied asynchronously into a two-stage ring -------------
#ifndef GEMM2M_RES_ROWS
#define GEMM2M_RES_ROWS 8
#endif
constexpr int kResRows = GEMM2M_RES_ROWS, kResK = 128, kResRun = 8, kResThreads = kResRows * kResK / kResRun;
constexpr int kResBlocksPerSm = 640 / kResThreads;   // 5 blocks of 128: up to 96 registers per thread measured faster than 6 blocks at 80
constexpr int kResIThreads = 256;
constexpr int kResRowStride = kResK + kResK / kResRun + 1;   // in elements: one pad per run of 8 + odd row stride -> no bank conflicts
constexpr int kResStages = 2;

template <typename T> struct RawCplx;
template <> struct RawCplx<double> { using type = double2; };
template <> struct RawCplx<float> { using type = float2; };

template <int BYTES>
__device__ __forceinline__ void cp_async_zfill(void* smem_dst, const void* gmem_src, bool valid) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const int src_bytes = valid ? BYTES : 0;   // 0 source bytes: the destination is filled with zeros
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;" ::"r"(d), "l"(gmem_src), "n"(BYTES), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <typename T, bool WIDE, int NMOD>
__global__ void __launch_bounds__(kResThreads, kResBlocksPerSm) residues_fp_kernel(const T* __restrict__ X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K,
                                                                     int64_t Kp, const int32_t* __restrict__ e,
                                                                     const __grid_constant__ ResidueTable tab, int8_t* __restrict__ planes) {
    using Raw = typename RawCplx<T>::type;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Raw* ring = reinterpret_cast<Raw*>(smem_raw);
    constexpr int kStageElems = kResRows * kResRowStride;
    const int t = threadIdx.x;
    const int64_t ktiles = Kp / kResK;
    const int64_t total = ((R + kResRows - 1) / kResRows) * ktiles;
    const int64_t plane_stride = R * Kp;

    auto issue = [&](int64_t tile, int stage) {
        const int64_t row0 = (tile / ktiles) * kResRows, k0 = (tile % ktiles) * kResK;
        Raw* dst = ring + stage * kStageElems;
        if (!k_contiguous) {          // consecutive threads -> consecutive operand rows (rows of a column-major matrix)
            const int r = t & (kResRows - 1);
            const int64_t row = row0 + r;
#pragma unroll
            for (int kk = t / kResRows; kk < kResK; kk += kResThreads / kResRows) {
                const int64_t k = k0 + kk;
                const bool ok = row < R && k < K;
                cp_async_zfill<sizeof(Raw)>(dst + r * kResRowStride + kk + (kk >> 3), ok ? X + 2 * (row + k * ld) : X, ok);
            }
        } else {                      // consecutive threads -> consecutive k (columns of the matrix are contiguous)
            const int kk = t & (kResK - 1);
            const int64_t k = k0 + kk;
#pragma unroll
            for (int r = t / kResK; r < kResRows; r += kResThreads / kResK) {
                const int64_t row = row0 + r;
                const bool ok = row < R && k < K;
                cp_async_zfill<sizeof(Raw)>(dst + r * kResRowStride + kk + (kk >> 3), ok ? X + 2 * (k + row * ld) : X, ok);
            }
        }
        cp_async_commit();
    };

    int64_t tile = blockIdx.x;
    if (tile >= total) return;
    issue(tile, 0);
    for (int it = 0; tile < total; tile += gridDim.x, ++it) {
        const int64_t next = tile + gridDim.x;
        if (next < total) { issue(next, (it + 1) & 1); cp_async_wait_group<1>(); }
        else cp_async_wait_group<0>();
        __syncthreads();
        const Raw* src = ring + (it & 1) * kStageElems;
        const int64_t row0 = (tile / ktiles) * kResRows, k0 = (tile % ktiles) * kResK;
        const int g = t & (kResK / kResRun - 1), r = t / (kResK / kResRun);
        const int64_t row = row0 + r;
        if (row < R) {
            const int ex = __ldg(e + row);
            // Narrow mode, ordinary exponents: x 2^-e is an exact FP64 product (or underflows towards zero, where the
            // truncation is zero anyway) and its truncation to int64 is one conversion; |x 2^-e| < 2^62 by the scaling rule.
            const bool fast = !WIDE && ex > -1000 && ex < 1000;
            const double scale = __longlong_as_double((long long)(1023 - (fast ? ex : 0)) << 52);
            Digits dr[kResRun], di[kResRun];
            uint32_t tr[WIDE ? kResRun : 1], ti[WIDE ? kResRun : 1];
#pragma unroll
            for (int i = 0; i < kResRun; ++i) {
                Raw v = src[r * kResRowStride + kResRun * g + g + i];
                if (conj) v.y = -v.y;                         // conjugated operand: the imaginary part changes sign before quantisation
                if (WIDE) {
                    uint32_t lr = 0, li = 0;
                    long long ur = 0, ui = 0;
                    if (ex != kExpNonFinite) {
                        quantise_part_wide<T>(v.x, ex, &lr, &ur);
                        quantise_part_wide<T>(v.y, ex, &li, &ui);
                    }
                    dr[i] = split_digits_wide(lr, ur, &tr[i]);
                    di[i] = split_digits_wide(li, ui, &ti[i]);
                } else {
                    long long qr = 0, qi = 0;
                    if (fast) {
                        qr = __double2ll_rz((double)v.x * scale);
                        qi = __double2ll_rz((double)v.y * scale);
                    } else if (ex != kExpNonFinite) {
                        qr = quantise_part<T>(v.x, ex);
                        qi = quantise_part<T>(v.y, ex);
                    }
                    dr[i] = split_digits(qr);
                    di[i] = split_digits(qi);
                }
            }
            emit_run<kResRun, WIDE, NMOD>(dr, di, tr, ti, tab, planes + row * Kp + k0 + kResRun * g, plane_stride);
        }
        __syncthreads();   // everyone is done with this stage before it is refilled
    }
}

constexpr size_t kResSmemBytes(size_t elem) { return (size_t)kResStages * kResRows * kResRowStride * elem; }


template <typename T>
cudaError_t launch_residues_fp(const T* X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K, int64_t Kp, const int32_t* e,
                               const ResidueTable& tab, bool wide, int8_t* planes, cudaStream_t st, int* launches) {
    if (R <= 0 || Kp <= 0) return cudaSuccess;
    constexpr size_t smem = kResSmemBytes(2 * sizeof(T));
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(residues_fp_kernel<T, false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess) err = cudaFuncSetAttribute(residues_fp_kernel<T, true, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
#define GEMM2M_RES_ATTR(N) if (err == cudaSuccess) err = cudaFuncSetAttribute(residues_fp_kernel<T, false, N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        GEMM2M_RES_ATTR(7) GEMM2M_RES_ATTR(8) GEMM2M_RES_ATTR(14) GEMM2M_RES_ATTR(15) GEMM2M_RES_ATTR(16)
#undef GEMM2M_RES_ATTR
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    const int64_t total = ((R + kResRows - 1) / kResRows) * (Kp / kResK);
    const int64_t resident = (int64_t)cached_sm_count() * kResBlocksPerSm;
    const unsigned grid = (unsigned)(total < resident ? total : resident);
    // The modulus counts of the common use cases (7-8: single precision and the fastest settings, 14-16: double precision)
    // get a specialisation with the modulus loop unrolled: the per-modulus constants become constant-bank operands, which
    // saves two instructions per (element, modulus) -- 13 % of the kernel's time at 16 moduli.
    const int spec = (!wide && tab.n2 == tab.nmod) ? tab.nmod : 0;
    switch (spec) {
#define GEMM2M_RES_CASE(N) case N: residues_fp_kernel<T, false, N><<<grid, kResThreads, smem, st>>>(X, ld, k_contiguous, conj, R, K, Kp, e, tab, planes); break;
        GEMM2M_RES_CASE(7) GEMM2M_RES_CASE(8) GEMM2M_RES_CASE(14) GEMM2M_RES_CASE(15) GEMM2M_RES_CASE(16)
#undef GEMM2M_RES_CASE
        default:
            if (wide) residues_fp_kernel<T, true, 0><<<grid, kResThreads, smem, st>>>(X, ld, k_contiguous, conj, R, K, Kp, e, tab, planes);
            else residues_fp_kernel<T, false, 0><<<grid, kResThreads, smem, st>>>(X, ld, k_contiguous, conj, R, K, Kp, e, tab, planes);
    }
    ++*launches;
    return cudaGetLastError();
}

// ---- real floating-point inputs (real Ozaki-II scheme): one plane per modulus ---------------------------------------
template <int NE, bool WIDE>
__device__ __forceinline__ void emit_run_real(const Digits (&dr)[NE], const uint32_t* tr, const ResidueTable& tab, int8_t* dst, int64_t plane_stride) {
    const int nmod = tab.nmod;
#pragma unroll 1
    for (int j = 0; j < nmod; ++j) {
        const int neg_m = -tab.m[j], y0 = tab.magic[j];
        const float inv_m = tab.inv_m[j], cq = tab.cq[j];
        const uint32_t wl = tab.w_lo[j], wh = tab.w_hi[j], wt = WIDE ? tab.w_top[j] : 0u;
        uint32_t rw[NE / 4];
#pragma unroll
        for (int w = 0; w < NE / 4; ++w) {
            uint32_t br[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int i = 4 * w + b;
                int Ry = dp4a_ss(dr[i].hi, wh, dp4a_us(dr[i].lo, wl, y0));
                if (WIDE) Ry = dp4a_ss(tr[i], wt, Ry);
                br[b] = sym_reduce_one(Ry, neg_m, inv_m, cq);
            }
            rw[w] = pack4(br);
        }
        store_run<NE>(dst + (int64_t)j * plane_stride, rw);
    }
}

template <typename T, bool WIDE>
__global__ void __launch_bounds__(kResThreads, kResBlocksPerSm) residues_real_kernel(const T* __restrict__ X, int64_t ld, bool k_contiguous, int64_t R,
                                                                                   int64_t K, int64_t Kp, const int32_t* __restrict__ e,
                                                                                   const __grid_constant__ ResidueTable tab, int8_t* __restrict__ planes) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* ring = reinterpret_cast<T*>(smem_raw);
    constexpr int kStageElems = kResRows * kResRowStride;
    const int t = threadIdx.x;
    const int64_t ktiles = Kp / kResK;
    const int64_t total = ((R + kResRows - 1) / kResRows) * ktiles;
    const int64_t plane_stride = R * Kp;

    auto issue = [&](int64_t tile, int stage) {
        const int64_t row0 = (tile / ktiles) * kResRows, k0 = (tile % ktiles) * kResK;
        T* dst = ring + stage * kStageElems;
        if (!k_contiguous) {
            const int r = t & (kResRows - 1);
            const int64_t row = row0 + r;
#pragma unroll
            for (int kk = t / kResRows; kk < kResK; kk += kResThreads / kResRows) {
                const int64_t k = k0 + kk;
                const bool ok = row < R && k < K;
                cp_async_zfill<sizeof(T)>(dst + r * kResRowStride + kk + (kk >> 3), ok ? X + (row + k * ld) : X, ok);
            }
        } else {
            const int kk = t & (kResK - 1);
            const int64_t k = k0 + kk;
#pragma unroll
            for (int r = t / kResK; r < kResRows; r += kResThreads / kResK) {
                const int64_t row = row0 + r;
                const bool ok = row < R && k < K;
                cp_async_zfill<sizeof(T)>(dst + r * kResRowStride + kk + (kk >> 3), ok ? X + (k + row * ld) : X, ok);
            }
        }
        cp_async_commit();
    };

    int64_t tile = blockIdx.x;
    if (tile >= total) return;
    issue(tile, 0);
    for (int it = 0; tile < total; tile += gridDim.x, ++it) {
        const int64_t next = tile + gridDim.x;
        if (next < total) { issue(next, (it + 1) & 1); cp_async_wait_group<1>(); }
        else cp_async_wait_group<0>();
        __syncthreads();
        const T* src = ring + (it & 1) * kStageElems;
        const int64_t row0 = (tile / ktiles) * kResRows, k0 = (tile % ktiles) * kResK;
        const int g = t & (kResK / kResRun - 1), r = t / (kResK / kResRun);
        const int64_t row = row0 + r;
        if (row < R) {
            const int ex = __ldg(e + row);
            const bool fast = !WIDE && ex > -1000 && ex < 1000;
            const double scale = __longlong_as_double((long long)(1023 - (fast ? ex : 0)) << 52);
            Digits dr[kResRun];
            uint32_t tr[WIDE ? kResRun : 1];
#pragma unroll
            for (int i = 0; i < kResRun; ++i) {
                const T v = src[r * kResRowStride + kResRun * g + g + i];
                if (WIDE) {
                    uint32_t lr = 0;
                    long long ur = 0;
                    if (ex != kExpNonFinite) quantise_part_wide<T>(v, ex, &lr, &ur);
                    dr[i] = split_digits_wide(lr, ur, &tr[i]);
                } else {
                    long long qr = 0;
                    if (fast) qr = __double2ll_rz((double)v * scale);
                    else if (ex != kExpNonFinite) qr = quantise_part<T>(v, ex);
                    dr[i] = split_digits(qr);
                }
            }
            emit_run_real<kResRun, WIDE>(dr, tr, tab, planes + row * Kp + k0 + kResRun * g, plane_stride);
        }
        __syncthreads();
    }
}

template <typename T>
cudaError_t launch_residues_real(const T* X, int64_t ld, bool k_contiguous, int64_t R, int64_t K, int64_t Kp, const int32_t* e,
                                 const ResidueTable& tab, bool wide, int8_t* planes, cudaStream_t st, int* launches) {
    if (R <= 0 || Kp <= 0) return cudaSuccess;
    constexpr size_t smem = kResSmemBytes(sizeof(T));
    const int64_t total = ((R + kResRows - 1) / kResRows) * (Kp / kResK);
    const int64_t resident = (int64_t)cached_sm_count() * kResBlocksPerSm;
    const unsigned grid = (unsigned)(total < resident ? total : resident);
    if (wide) residues_real_kernel<T, true><<<grid, kResThreads, smem, st>>>(X, ld, k_contiguous, R, K, Kp, e, tab, planes);
    else residues_real_kernel<T, false><<<grid, kResThreads, smem, st>>>(X, ld, k_contiguous, R, K, Kp, e, tab, planes);
    ++*launches;
    return cudaGetLastError();
}
template cudaError_t launch_residues_real<double>(const double*, int64_t, bool, int64_t, int64_t, int64_t, const int32_t*, const ResidueTable&, bool, int8_t*, cudaStream_t, int*);

// ---- int8 Gaussian-integer inputs (no scaling): one 32 x 128 tile per block, loaded synchronously ---------------------
constexpr int kResIRows = 32, kResIRun = 16;
constexpr int kResIRowStride = kResK + kResK / kResIRun + 1;

__global__ void __launch_bounds__(kResIThreads) residues_int8_kernel(const int8_t* __restrict__ Xr, const int8_t* __restrict__ Xi, int64_t ld,
                                                                    bool k_contiguous, int64_t R, int64_t K, int64_t Kp,
                                                                    const __grid_constant__ ResidueTable tab, int8_t* __restrict__ planes) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    QPair* tile = reinterpret_cast<QPair*>(smem_raw);
    const int64_t row0 = (int64_t)blockIdx.y * kResIRows, k0 = (int64_t)blockIdx.x * kResK;
    const int t = threadIdx.x;
    auto fetch = [&](int r, int kk) -> QPair {
        const int64_t row = row0 + r, k = k0 + kk;
        QPair q{0, 0};
        if (row < R && k < K) {
            const int64_t idx = k_contiguous ? k + row * ld : row + k * ld;
            q.re = Xr[idx];
            q.im = Xi[idx];
        }
        return q;
    };
    if (!k_contiguous) {
        const int r = t & 31;
        for (int kk = t >> 5; kk < kResK; kk += kResIThreads / 32) tile[r * kResIRowStride + kk + (kk >> 4)] = fetch(r, kk);
    } else {
        const int kk = t & (kResK - 1);
        for (int r = t >> 7; r < kResIRows; r += kResIThreads / kResK) tile[r * kResIRowStride + kk + (kk >> 4)] = fetch(r, kk);
    }
    __syncthreads();
    const int g = t & 7, r = t >> 3;
    Digits dr[kResIRun], di[kResIRun];
#pragma unroll
    for (int i = 0; i < kResIRun; ++i) {
        const QPair q = tile[r * kResIRowStride + kResIRun * g + i + g];
        dr[i] = split_digits(q.re);
        di[i] = split_digits(q.im);
    }
    const int64_t row = row0 + r;
    if (row >= R) return;
    emit_run<kResIRun, false, 0>(dr, di, nullptr, nullptr, tab, planes + row * Kp + k0 + kResIRun * g, R * Kp);
}

cudaError_t launch_residues_int8(const int8_t* Xr, const int8_t* Xi, int64_t ld, bool k_contiguous, int64_t R, int64_t K, int64_t Kp,
                                 const ResidueTable& tab, int8_t* planes, cudaStream_t st, int* launches) {
    if (R <= 0 || Kp <= 0) return cudaSuccess;
    constexpr size_t smem = (size_t)kResIRows * kResIRowStride * sizeof(QPair);
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(residues_int8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    dim3 grid((unsigned)(Kp / kResK), (unsigned)((R + kResIRows - 1) / kResIRows));
    residues_int8_kernel<<<grid, kResIThreads, smem, st>>>(Xr, Xi, ld, k_contiguous, R, K, Kp, tab, planes);
    ++*launches;
    return cudaGetLastError();
}

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
    for (int c = 0; c < NCH; ++c) S[c] = fma(-t, tab.Mc[c], S[c]);          // exact: |t| < 2^12, digits < 2^40
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

__device__ __forceinline__ double scale_pow2(double x, int e) {   // x 2^e with e split so that both factors are normal
    const int e1 = max(-1000, min(1000, e));
    const int e2 = max(-1000, min(1000, e - e1));
    const int e3 = e - e1 - e2;
    double y = x * __longlong_as_double((long long)(e1 + 1023) << 52);
    if (e2) y *= __longlong_as_double((long long)(e2 + 1023) << 52);
    if (e3) y = ldexp(y, e3);
    return y;
}

template <typename T> __device__ __forceinline__ void store4(T* dst, const double (&re)[4], const double (&im)[4], int count);
template <> __device__ __forceinline__ void store4<double>(double* dst, const double (&re)[4], const double (&im)[4], int count) {
    for (int i = 0; i < count; ++i) *reinterpret_cast<double2*>(dst + 2 * i) = make_double2(re[i], im[i]);
}
template <> __device__ __forceinline__ void store4<float>(float* dst, const double (&re)[4], const double (&im)[4], int count) {
    if (count == 4 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
        *reinterpret_cast<float4*>(dst) = make_float4((float)re[0], (float)im[0], (float)re[1], (float)im[1]);
        *reinterpret_cast<float4*>(dst + 4) = make_float4((float)re[2], (float)im[2], (float)re[3], (float)im[3]);
    } else {
        for (int i = 0; i < count; ++i) *reinterpret_cast<float2*>(dst + 2 * i) = make_float2((float)re[i], (float)im[i]);
    }
}

constexpr int kPostThreads = 128;
constexpr int kPostSpan = kPostThreads * 4;   // consecutive row indices i handled by one block

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// cpm: [planes][n][ldp] int8 (row index i contiguous), planes = C+ and C- of the 2M moduli, then P1, P2, P3 of the 3M
// moduli.  A block handles 512 consecutive i of one column j: it first pulls the planes x 512 residue bytes into shared memory with asynchronous 16-byte copies (all in flight at once), then each
// thread combines 4 consecutive i.
// AXPBY: C = alpha X + beta C (alpha, beta complex, given as re/im pairs) instead of C = X; the product X is formed
// exactly as before, then combined in FP64 with fused multiply-adds.  beta = 0 does not read C.
struct PostScalars { double ar, ai, br, bi; };

template <typename T, int NCH, bool AXPBY>
__global__ void __launch_bounds__(kPostThreads) post_fp_kernel(const int8_t* __restrict__ cpm, int64_t ldp, int64_t m, int64_t n,
                                                               const int32_t* __restrict__ eA, const int32_t* __restrict__ eB,
                                                               const __grid_constant__ CrtTable tab, T* __restrict__ C, int64_t ldc,
                                                               const PostScalars sc) {
    __shared__ __align__(16) uint32_t stage[kMaxPlanes][kPostThreads];
    const int64_t ib = (int64_t)blockIdx.x * kPostSpan;
    const int64_t j = blockIdx.y;
    const int nmod = tab.nmod, n2 = tab.n2, n3 = nmod - n2;
    const int64_t plane = n * ldp;
    const int8_t* src = cpm + j * ldp + ib;
    const int vec_per_plane = (int)min((int64_t)(kPostSpan / 16), (ldp - ib) / 16);   // ldp is a multiple of 16
    for (int idx = threadIdx.x; idx < (2 * n2 + 3 * n3) * (kPostSpan / 16); idx += kPostThreads) {
        const int p = idx / (kPostSpan / 16), v = idx - p * (kPostSpan / 16);
        if (v < vec_per_plane) cp_async16(&stage[p][4 * v], src + (int64_t)p * plane + 16 * v);
    }
    cp_async_wait_all();
    __syncthreads();
    const int64_t i0 = ib + 4 * threadIdx.x;
    if (i0 >= m) return;
    double Sr[4][NCH], Si[4][NCH];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
#pragma unroll
        for (int c = 0; c < NCH; ++c) Sr[e][c] = Si[e][c] = 0.0;
    }
#pragma unroll 2
    for (int jm = 0; jm < n2; ++jm) {
        const uint32_t wp = stage[jm][threadIdx.x];            // c+ of 4 elements
        const uint32_t wm = stage[n2 + jm][threadIdx.x];       // c-
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int cp = sbyte(wp, e);
            const int cm = sbyte(wm, e);
            const double vr = int_to_double(cm + cp);     // Eq. (2c): real part uses C- + C+
            const double vi = int_to_double(cm - cp);     //           imaginary part uses C- - C+
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                Sr[e][c] = fma(vr, tab.gr[jm][c], Sr[e][c]);
                Si[e][c] = fma(vi, tab.gi[jm][c], Si[e][c]);
            }
        }
    }
#pragma unroll 1
    for (int j3 = 0; j3 < n3; ++j3) {                      // 3M moduli of the hybrid, Eq. (1)
        const uint32_t w1 = stage[2 * n2 + j3][threadIdx.x];
        const uint32_t w2 = stage[2 * n2 + n3 + j3][threadIdx.x];
        const uint32_t w3 = stage[2 * n2 + 2 * n3 + j3][threadIdx.x];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int p1 = sbyte(w1, e), p2 = sbyte(w2, e), p3 = sbyte(w3, e);
            const double vr = int_to_double(p1 - p2);
            const double vi = int_to_double(p3 - p1 - p2);
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                Sr[e][c] = fma(vr, tab.gr[n2 + j3][c], Sr[e][c]);
                Si[e][c] = fma(vi, tab.gr[n2 + j3][c], Si[e][c]);
            }
        }
    }
    const int fb = __ldg(eB + j);
    double re[4], im[4];
    int count = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        if (i0 + e < m) {
            ++count;
            const int ea = __ldg(eA + i0 + e);
            if (ea == kExpNonFinite || fb == kExpNonFinite) {
                re[e] = im[e] = __longlong_as_double(0x7FF8000000000000ll);
            } else {
                double h, l;
                crt_finish<NCH>(Sr[e], tab, &h, &l);
                re[e] = scale_pow2(h + l, ea + fb);
                crt_finish<NCH>(Si[e], tab, &h, &l);
                im[e] = scale_pow2(h + l, ea + fb);
            }
        }
    }
    if (AXPBY) {
        const bool use_c = sc.br != 0.0 || sc.bi != 0.0;
        for (int e = 0; e < count; ++e) {
            const double xr = re[e], xi = im[e];
            double yr = fma(sc.ar, xr, -sc.ai * xi), yi = fma(sc.ar, xi, sc.ai * xr);
            if (use_c) {
                const T* old = C + 2 * (i0 + e + j * ldc);
                const double cr = (double)old[0], ci = (double)old[1];
                yr += fma(sc.br, cr, -sc.bi * ci);
                yi += fma(sc.br, ci, sc.bi * cr);
            }
            re[e] = yr;
            im[e] = yi;
        }
    }
    store4<T>(C + 2 * (i0 + j * ldc), re, im, count);
}

template <typename T, bool AXPBY>
static cudaError_t launch_post_fp_t(const int8_t* cpm, int64_t ldp, int64_t m, int64_t n, int64_t j_begin, int64_t j_end, const int32_t* eA,
                                    const int32_t* eB, const CrtTable& tab, T* C, int64_t ldc, const PostScalars& sc, cudaStream_t st,
                                    int* launches) {
    const int64_t per_block = kPostSpan;
    for (int64_t j0 = j_begin; j0 < j_end; j0 += 65535) {      // grid.y limit
        const int64_t nj = (j_end - j0 < 65535) ? j_end - j0 : 65535;
        dim3 grid((unsigned)((m + per_block - 1) / per_block), (unsigned)nj);
        const int8_t* src = cpm + j0 * ldp;
        T* dst = C + 2 * j0 * ldc;
        // the plane stride is n * ldp for the whole matrix, so pass the full n and offset pointers
        switch (tab.nchunks) {
            case 1: post_fp_kernel<T, 1, AXPBY><<<grid, kPostThreads, 0, st>>>(src, ldp, m, n, eA, eB + j0, tab, dst, ldc, sc); break;
            case 2: post_fp_kernel<T, 2, AXPBY><<<grid, kPostThreads, 0, st>>>(src, ldp, m, n, eA, eB + j0, tab, dst, ldc, sc); break;
            case 3: post_fp_kernel<T, 3, AXPBY><<<grid, kPostThreads, 0, st>>>(src, ldp, m, n, eA, eB + j0, tab, dst, ldc, sc); break;
            case 4: post_fp_kernel<T, 4, AXPBY><<<grid, kPostThreads, 0, st>>>(src, ldp, m, n, eA, eB + j0, tab, dst, ldc, sc); break;
            default: post_fp_kernel<T, 5, AXPBY><<<grid, kPostThreads, 0, st>>>(src, ldp, m, n, eA, eB + j0, tab, dst, ldc, sc); break;
        }
        ++*launches;
    }
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_post_fp(const int8_t* cpm, int64_t ldp, int64_t m, int64_t n, int64_t j_begin, int64_t j_end, const int32_t* eA,
                           const int32_t* eB, const CrtTable& tab, T* C, int64_t ldc, const double* alpha, const double* beta,
                           cudaStream_t st, int* launches) {
    if (m <= 0 || j_end <= j_begin) return cudaSuccess;
    PostScalars sc{1.0, 0.0, 0.0, 0.0};
    if (alpha) { sc.ar = alpha[0]; sc.ai = alpha[1]; }
    if (beta) { sc.br = beta[0]; sc.bi = beta[1]; }
    const bool plain = sc.ar == 1.0 && sc.ai == 0.0 && sc.br == 0.0 && sc.bi == 0.0;
    if (plain) return launch_post_fp_t<T, false>(cpm, ldp, m, n, j_begin, j_end, eA, eB, tab, C, ldc, sc, st, launches);
    return launch_post_fp_t<T, true>(cpm, ldp, m, n, j_begin, j_end, eA, eB, tab, C, ldc, sc, st, launches);
}

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

// HERK (Section 5): only C+ = A+ A-^T was computed; C- = C+^T.  cp: [nmod][n][ldp] with cp[j][col][row] = C+_j[row, col].
// A block handles 64 rows i x 16 columns j of the lower triangle.  It needs C+[i, j] (rows of cp along i: 16 runs of 64
// bytes per modulus) and C-[i, j] = C+[j, i] (rows of cp along j: 64 runs of 16 bytes per modulus); both are pulled into
// shared memory with asynchronous 16-byte copies, then each thread combines 4 consecutive i of one column.
// Lower triangle only; on the diagonal C- - C+ = 0, so the imaginary part is exactly zero.
constexpr int kHerkI = 64, kHerkJ = 16, kHerkThreads = 256;
constexpr int kHerkMirrorSlots = kHerkI + kHerkI / 8;                      // 16-byte slots, one pad slot per 8 rows (bank spread)
constexpr int kHerkPlaneBytes = kHerkJ * kHerkI + kHerkMirrorSlots * 16;   // direct + mirrored bytes per modulus

template <int NCH, bool REAL_OUT>
__global__ void __launch_bounds__(kHerkThreads) post_herk_kernel(const int8_t* __restrict__ cp, int64_t ldp, int64_t n, int64_t i_begin,
                                                                 const int32_t* __restrict__ eA, const __grid_constant__ CrtTable tab,
                                                                 double* __restrict__ C, int64_t ldc) {
    extern __shared__ __align__(16) unsigned char herk_smem[];
    const int64_t ibase = i_begin + (int64_t)blockIdx.x * kHerkI, jbase = (int64_t)blockIdx.y * kHerkJ;
    if (ibase + kHerkI - 1 < jbase) return;                                // tile entirely above the diagonal
    const int nmod = tab.nmod;
    const int64_t plane = n * ldp;
    const int t = threadIdx.x;
    // direct part: for each modulus and each column j of the tile, 64 bytes along i (4 copies of 16 bytes)
    for (int idx = t; idx < nmod * kHerkJ * (kHerkI / 16); idx += kHerkThreads) {
        const int v = idx & 3, jj = (idx >> 2) & (kHerkJ - 1), jm = idx / (kHerkJ * 4);
        const int64_t i = ibase + 16 * v, j = jbase + jj;
        if (j < n && i < ldp) cp_async16(herk_smem + jm * kHerkPlaneBytes + jj * kHerkI + 16 * v, cp + (int64_t)jm * plane + j * ldp + i);
    }
    // mirrored part: for each modulus and each row i of the tile, the 16 bytes C+[jbase .. jbase+15, i]
    for (int idx = t; idx < nmod * kHerkI; idx += kHerkThreads) {
        const int ii = idx & (kHerkI - 1), jm = idx / kHerkI;
        const int64_t i = ibase + ii;
        if (i < n && jbase < ldp)
            cp_async16(herk_smem + jm * kHerkPlaneBytes + kHerkJ * kHerkI + (ii + (ii >> 3)) * 16, cp + (int64_t)jm * plane + i * ldp + jbase);
    }
    cp_async_wait_all();
    __syncthreads();
    const int g = t & 15, jj = t >> 4;                                     // 4 consecutive rows i0 .. i0+3 of column j
    const int64_t i0 = ibase + 4 * g, j = jbase + jj;
    if (j >= n || i0 >= n || i0 + 3 < j) return;
    double Sr[4][NCH], Si[4][NCH];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
#pragma unroll
        for (int c = 0; c < NCH; ++c) Sr[e][c] = Si[e][c] = 0.0;
    }
#pragma unroll 2
    for (int jm = 0; jm < nmod; ++jm) {
        const unsigned char* base = herk_smem + jm * kHerkPlaneBytes;
        const uint32_t wp = *reinterpret_cast<const uint32_t*>(base + jj * kHerkI + 4 * g);      // C+[i0..i0+3, j]
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int ii = 4 * g + e;
            const int cpv = sbyte(wp, e);
            const int cmv = (int)(int8_t)base[kHerkJ * kHerkI + (ii + (ii >> 3)) * 16 + jj];    // C-[i, j] = C+[j, i]
            const double vr = int_to_double(cmv + cpv), vi = int_to_double(cmv - cpv);
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                Sr[e][c] = fma(vr, tab.gr[jm][c], Sr[e][c]);
                if (!REAL_OUT) Si[e][c] = fma(vi, tab.gi[jm][c], Si[e][c]);
            }
        }
    }
    const int ej = __ldg(eA + j);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int64_t i = i0 + e;
        if (i < n && i >= j) {
            const int ei = __ldg(eA + i);
            double re, im = 0.0;
            if (ei == kExpNonFinite || ej == kExpNonFinite) {
                re = im = __longlong_as_double(0x7FF8000000000000ll);
            } else {
                double h, l;
                crt_finish<NCH>(Sr[e], tab, &h, &l);
                re = scale_pow2(h + l, ei + ej);
                if (!REAL_OUT) {
                    crt_finish<NCH>(Si[e], tab, &h, &l);
                    im = scale_pow2(h + l, ei + ej);
                }
            }
            if (REAL_OUT) C[i + j * ldc] = re;
            else *reinterpret_cast<double2*>(C + 2 * (i + j * ldc)) = make_double2(re, im);
        }
    }
}

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

template <bool REAL_OUT>
static cudaError_t launch_post_herk_t(const int8_t* cp, int64_t ldp, int64_t n, int64_t i_begin, int64_t i_end, const int32_t* eA,
                                      const CrtTable& tab, double* C, int64_t ldc, cudaStream_t st, int* launches) {
    const size_t smem = (size_t)kMaxMod * kHerkPlaneBytes;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(post_herk_kernel<1, REAL_OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess) err = cudaFuncSetAttribute(post_herk_kernel<2, REAL_OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess) err = cudaFuncSetAttribute(post_herk_kernel<3, REAL_OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess) err = cudaFuncSetAttribute(post_herk_kernel<4, REAL_OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    const size_t use = (size_t)tab.nmod * kHerkPlaneBytes;
    const int64_t tiles_j = (i_end + kHerkJ - 1) / kHerkJ;  // lower triangle: columns up to the last row of the range
    if (tiles_j > 65535) return cudaErrorInvalidValue;     // n beyond 65535 * 16 columns: far beyond any workspace
    dim3 grid((unsigned)((i_end - i_begin + kHerkI - 1) / kHerkI), (unsigned)tiles_j);
    switch (tab.nchunks) {
        case 1: post_herk_kernel<1, REAL_OUT><<<grid, kHerkThreads, use, st>>>(cp, ldp, n, i_begin, eA, tab, C, ldc); break;
        case 2: post_herk_kernel<2, REAL_OUT><<<grid, kHerkThreads, use, st>>>(cp, ldp, n, i_begin, eA, tab, C, ldc); break;
        case 3: post_herk_kernel<3, REAL_OUT><<<grid, kHerkThreads, use, st>>>(cp, ldp, n, i_begin, eA, tab, C, ldc); break;
        default: post_herk_kernel<4, REAL_OUT><<<grid, kHerkThreads, use, st>>>(cp, ldp, n, i_begin, eA, tab, C, ldc); break;
    }
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_post_herk(const int8_t* cp, int64_t ldp, int64_t n, int64_t i_begin, int64_t i_end, const int32_t* eA, const CrtTable& tab,
                             double* C, int64_t ldc, bool real_out, cudaStream_t st, int* launches) {
    if (n <= 0 || i_end <= i_begin) return cudaSuccess;
    return real_out ? launch_post_herk_t<true>(cp, ldp, n, i_begin, i_end, eA, tab, C, ldc, st, launches)
                    : launch_post_herk_t<false>(cp, ldp, n, i_begin, i_end, eA, tab, C, ldc, st, launches);
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

// explicit instantiations
template cudaError_t launch_scan_rows<double>(const double*, int64_t, int64_t, int64_t, uint64_t*, cudaStream_t, int*);
template cudaError_t launch_scan_rows<float>(const float*, int64_t, int64_t, int64_t, uint64_t*, cudaStream_t, int*);
template cudaError_t launch_scan_cols<double>(const double*, int64_t, int64_t, int64_t, uint64_t*, cudaStream_t, int*);
template cudaError_t launch_scan_cols<float>(const float*, int64_t, int64_t, int64_t, uint64_t*, cudaStream_t, int*);
template cudaError_t launch_exponents<double>(const uint64_t*, int64_t, int, int, int32_t*, cudaStream_t, int*);
template cudaError_t launch_exponents<float>(const uint64_t*, int64_t, int, int, int32_t*, cudaStream_t, int*);
template cudaError_t launch_residues_fp<double>(const double*, int64_t, bool, bool, int64_t, int64_t, int64_t, const int32_t*, const ResidueTable&, bool, int8_t*, cudaStream_t, int*);
template cudaError_t launch_residues_fp<float>(const float*, int64_t, bool, bool, int64_t, int64_t, int64_t, const int32_t*, const ResidueTable&, bool, int8_t*, cudaStream_t, int*);
template cudaError_t launch_post_fp<double>(const int8_t*, int64_t, int64_t, int64_t, int64_t, int64_t, const int32_t*, const int32_t*, const CrtTable&, double*, int64_t, const double*, const double*, cudaStream_t, int*);
template cudaError_t launch_post_fp<float>(const int8_t*, int64_t, int64_t, int64_t, int64_t, int64_t, const int32_t*, const int32_t*, const CrtTable&, float*, int64_t, const double*, const double*, cudaStream_t, int*);

}  // namespace gemm2m

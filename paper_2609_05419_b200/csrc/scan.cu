// Algorithm 1 step 2: exponent scans and scale exponents (largest-part rule, 2-norm rule), for complex and real matrices.
// Streaming kernels bounded by HBM bandwidth.
#include "prepost_common.cuh"

namespace gemm2m {

// =====================================================================================================
// Step 2: exponent scan.  For every row (or column) the largest magnitude bit pattern of any real or
// imaginary part; IEEE bit patterns of non-negative numbers are ordered like the numbers themselves.
// =====================================================================================================
constexpr int kScanThreads = 256;
constexpr int kScanRowsSpan = 64;     // columns handled by one block of scan_rows
constexpr int kScanColsSpan = 2048;   // rows handled by one warp of scan_cols

// One thread per row, a span of columns per block: consecutive threads read consecutive rows (coalesced).
template <typename T>
__global__ void __launch_bounds__(kScanThreads) scan_rows_kernel(const T* __restrict__ X, int64_t rows, int64_t cols, int64_t ld, int64_t span,
                                                                 unsigned long long* __restrict__ absmax) {
    wait_for_prior_kernels();
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
    wait_for_prior_kernels();
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
    e[i] = scale_exponent<T>(absmax[i], P, ck);
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
cudaError_t launch_scan_rows(const T* X, int64_t rows, int64_t cols, int64_t ld, uint64_t* absmax, cudaStream_t st, int* launches, bool chained) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    int64_t span = kScanRowsSpan;
    const int64_t row_blocks = (rows + kScanThreads - 1) / kScanThreads;
    while (span > 8 && row_blocks * ((cols + span - 1) / span) < 4 * cached_sm_count()) span /= 2;   // small matrices: enough blocks to fill the GPU
    while ((cols + span - 1) / span > 65535) span *= 2;        // grid.y limit
    dim3 grid((unsigned)row_blocks, (unsigned)((cols + span - 1) / span));
    if (chained) launch_chained(scan_rows_kernel<T>, grid, dim3(kScanThreads), 0, st, X, rows, cols, ld, span, (unsigned long long*)absmax);
    else scan_rows_kernel<T><<<grid, kScanThreads, 0, st>>>(X, rows, cols, ld, span, (unsigned long long*)absmax);
    ++*launches;
    return cudaGetLastError();
}
template <typename T>
cudaError_t launch_scan_cols(const T* X, int64_t rows, int64_t cols, int64_t ld, uint64_t* absmax, cudaStream_t st, int* launches, bool chained) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    int64_t span = kScanColsSpan;
    const int64_t col_blocks = (cols + kScanThreads / 32 - 1) / (kScanThreads / 32);
    while (span > 256 && col_blocks * ((rows + span - 1) / span) < 4 * cached_sm_count()) span /= 2;
    while ((rows + span - 1) / span > 65535) span *= 2;        // grid.y limit
    dim3 grid((unsigned)col_blocks, (unsigned)((rows + span - 1) / span));
    if (chained) launch_chained(scan_cols_kernel<T>, grid, dim3(kScanThreads), 0, st, X, rows, cols, ld, span, (unsigned long long*)absmax);
    else scan_cols_kernel<T><<<grid, kScanThreads, 0, st>>>(X, rows, cols, ld, span, (unsigned long long*)absmax);
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

template cudaError_t launch_scan_rows<double>(const double*, int64_t, int64_t, int64_t, uint64_t*, cudaStream_t, int*, bool);
template cudaError_t launch_scan_rows<float>(const float*, int64_t, int64_t, int64_t, uint64_t*, cudaStream_t, int*, bool);
template cudaError_t launch_scan_cols<double>(const double*, int64_t, int64_t, int64_t, uint64_t*, cudaStream_t, int*, bool);
template cudaError_t launch_scan_cols<float>(const float*, int64_t, int64_t, int64_t, uint64_t*, cudaStream_t, int*, bool);
template cudaError_t launch_exponents<double>(const uint64_t*, int64_t, int, int, int32_t*, cudaStream_t, int*);
template cudaError_t launch_exponents<float>(const uint64_t*, int64_t, int, int, int32_t*, cudaStream_t, int*);

}  // namespace gemm2m

// Pieces shared by the residue kernels (Algorithm 1 steps 3 + 4): truncating quantisation of one part, and the staging of raw
// operand tiles in shared memory with asynchronous copies.
#pragma once
#include "prepost_common.cuh"

namespace gemm2m {

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

}  // namespace gemm2m

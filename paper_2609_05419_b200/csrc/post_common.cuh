// Device helpers shared by the post-processing kernels (Algorithm 1 steps 4-7).
#pragma once
#include "prepost_common.cuh"

namespace gemm2m {

__device__ __forceinline__ double scale_pow2(double x, int e) {   // x 2^e with e split so that both factors are normal
    const int e1 = max(-1000, min(1000, e));
    const int e2 = max(-1000, min(1000, e - e1));
    const int e3 = e - e1 - e2;
    double y = x * __longlong_as_double((long long)(e1 + 1023) << 52);
    if (e2) y *= __longlong_as_double((long long)(e2 + 1023) << 52);
    if (e3) y = ldexp(y, e3);
    return y;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void cp_async_commit_group() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait_pending() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// C = alpha X + beta C (alpha, beta complex, given as re/im pairs) instead of C = X: the product X is formed and rounded
// first, then combined in FP64 with fused multiply-adds.  beta = 0 does not read C.
struct PostScalars { double ar, ai, br, bi; };

}  // namespace gemm2m

// Plain CUDA-core int8 GEMM with the same contract as the tcgen05 kernel (Eq. 2b): out = sym(rowop colop^T mod m_j) per batch
// entry.  Kept only so that tests can tell a fault in the tensor-core kernel from one in the pre/post kernels.
#include "gemm_ptx.cuh"

namespace gemm2m {

// ------------------------------------------------------------------------------------------------ check kernel
// Plain CUDA-core version of the same contract (one thread per output entry, dp4a over K).  Only for tests.
__global__ void __launch_bounds__(256) gemm_i8_check_kernel(const int8_t* __restrict__ rowop, const int8_t* __restrict__ colop, int64_t R,
                                                            int64_t Cn, int64_t Kp, int64_t k_chunk, int row_plane0, int col_plane0,
                                                            int8_t* __restrict__ out, int64_t ldp, const __grid_constant__ ModTable mods,
                                                            int64_t row_begin, int64_t row_end, int accumulate) {
    const int64_t c = (int64_t)blockIdx.x * 16 + (threadIdx.x & 15);
    const int64_t r = row_begin + (int64_t)blockIdx.y * 16 + (threadIdx.x >> 4);
    const int b = blockIdx.z;
    if (r >= R || r >= row_end || c >= Cn) return;
    const int jm = b;
    const int m = mods.m[jm];
    const int* pr = reinterpret_cast<const int*>(rowop + ((int64_t)(row_plane0 + b) * R + r) * Kp);
    const int* pc = reinterpret_cast<const int*>(colop + ((int64_t)(col_plane0 + b) * Cn + c) * Kp);
    int res = accumulate ? (int)out[(int64_t)b * R * ldp + r * ldp + c] : 0;
    for (int64_t k0 = 0; k0 < Kp; k0 += k_chunk) {
        const int64_t k1 = (k0 + k_chunk < Kp) ? k0 + k_chunk : Kp;
        int acc = 0;
        for (int64_t k = k0 / 4; k < k1 / 4; ++k) acc = __dp4a(pr[k], pc[k], acc);
        res = (res + acc % m) % m;
    }
    if (res > (m - 1) / 2) res -= m; else if (res < -(m / 2)) res += m;   // [-(m-1)/2, (m-1)/2]; even m: [-m/2, m/2 - 1]
    out[(int64_t)b * R * ldp + r * ldp + c] = (int8_t)res;
}

cudaError_t launch_gemm_check(const GemmArgs& a, int64_t k_limit, cudaStream_t st, int* launches) {
    if (a.R <= 0 || a.Cn <= 0 || a.nbatch <= 0 || a.row_end <= a.row_begin) return cudaSuccess;
    int64_t chunk = (k_limit / kGemmBK) * kGemmBK;
    if (chunk <= 0) chunk = kGemmBK;
    dim3 grid((unsigned)((a.Cn + 15) / 16), (unsigned)((a.row_end - a.row_begin + 15) / 16), (unsigned)a.nbatch);
    gemm_i8_check_kernel<<<grid, 256, 0, st>>>(a.rowop, a.colop, a.R, a.Cn, a.Kp, chunk, a.row_plane0, a.col_plane0, a.out, a.ldp, a.mods,
                                               a.row_begin, a.row_end, a.accumulate);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace gemm2m

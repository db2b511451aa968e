// Batched int8 GEMM with modular epilogue, Eq. (2b): C+- = A+- B+- (mod m_j), on the 5th-generation tensor cores.
//
// One persistent CTA per SM walks over (batch, tile) pairs.  Warp roles:
//   warp 0      TMA producer: loads 128-byte-wide K slices of both operands (128B swizzle) into a shared-memory ring
//   warp 1      MMA issuer: tcgen05.mma.kind::i8 (128 x 256 x 32 per instruction), int32 accumulators in TMEM,
//               two accumulator buffers so that the epilogue of one tile overlaps the MMAs of the next
//   warps 2-5   epilogue: tcgen05.ld the accumulators, reduce each exactly modulo m_j to the symmetric residue and
//               store one byte per entry (the int32 products never travel to HBM)
// int32 accumulation is exact as long as K ((m-1)/2)^2 < 2^31; the host splits K beyond that and the epilogue adds
// the residue already stored (accumulate flag).
// Every wait on an mbarrier is bounded in time; on a timeout the kernel records a code in the status word, all
// roles leave their loops, TMEM is released and the kernel returns.
#include "gemm_ptx.cuh"

namespace gemm2m {

namespace cfg {
constexpr int BM = 128;        // TMEM lanes: rows of the "row operand" per tile
constexpr int BN = 256;        // TMEM columns: rows of the "column operand" per tile
constexpr int BK = 128;        // bytes (= int8 elements) of K per pipeline stage: one 128-byte swizzle row
constexpr int UMMA_K = 32;     // K of one tcgen05.mma.kind::i8
constexpr int STAGES = 4;
constexpr int ROW_TILE_BYTES = BM * BK;   // 16 KB
constexpr int COL_TILE_BYTES = BN * BK;   // 32 KB
constexpr int STAGE_BYTES = ROW_TILE_BYTES + COL_TILE_BYTES;
constexpr int THREADS = 192;
constexpr int TMEM_COLS = 512; // two accumulators of 256 columns
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
}  // namespace cfg

__global__ void __launch_bounds__(cfg::THREADS, 1)
gemm_i8_tcgen05_kernel(const __grid_constant__ CUtensorMap map_row, const __grid_constant__ CUtensorMap map_col,
                       const __grid_constant__ GemmKernelParams p) {
    using namespace cfg;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;                      // 128B-swizzle atoms need 1024-byte alignment
    unsigned char* gen_base = smem_raw + (tiles_base - raw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + (size_t)STAGES * STAGE_BYTES);
    // barrier slots: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]; then tmem base (u32) and abort flag (int)
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES, bar_tempty = bar_tfull + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull + 8 * a, 1); mbar_init(bar_tempty + 8 * a, 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // TMEM allocation by one full warp
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int tiles_per_batch = p.tiles_r * p.tiles_c;
    const int total_tiles = tiles_per_batch * p.nbatch;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
                int b, tr, tc;
                decode_tile(p, tile, &b, &tr, &tc);
                for (int kb = 0; kb < p.kblocks; ++kb) {
                    if (!(ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, kDevTimeoutProducer))) break;
                    const uint32_t dst = tiles_base + stage * STAGE_BYTES;
                    mbar_arrive_expect_tx(bar_full + 8 * stage, STAGE_BYTES);
                    const int x = (p.kblock0 + kb) * BK;
                    tma_load_3d(dst, &map_row, bar_full + 8 * stage, x, tr * BM, p.row_plane0 + b);
                    tma_load_3d(dst + ROW_TILE_BYTES, &map_col, bar_full + 8 * stage, x, tc * BN, p.col_plane0 + b);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // gave up: let the copies already in flight land before the CTA's shared memory goes away
                for (int s = 0; s < STAGES; ++s) {
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(bar_full + 8 * s, 0) && !mbar_try_wait(bar_full + 8 * s, 1) &&
                           global_timer_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_i8(BM, BN);
            uint32_t stage = 0, phase = 0;
            uint32_t acc_phase[2] = {0, 0};
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++it) {
                const int acc = it & 1;
                if (!(ok = mbar_wait(bar_tempty + 8 * acc, acc_phase[acc] ^ 1u, abort_flag, p.dev_status, kDevTimeoutMma))) break;
                acc_phase[acc] ^= 1u;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < p.kblocks; ++kb) {
                    if (!(ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.dev_status, kDevTimeoutMma))) break;
                    tcgen05_fence_after();
                    const uint32_t a_addr = tiles_base + stage * STAGE_BYTES;
                    const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(a_addr + ROW_TILE_BYTES);
#pragma unroll
                    for (int k4 = 0; k4 < BK / UMMA_K; ++k4) {
                        // advancing K inside the swizzled 128-byte row: +32 bytes = +2 in the 16-byte address field
                        umma_i8(d_tmem, adesc + (uint64_t)(k4 * (UMMA_K >> 4)), bdesc + (uint64_t)(k4 * (UMMA_K >> 4)), idesc,
                                (uint32_t)((kb | k4) != 0));
                    }
                    umma_commit(bar_empty + 8 * stage);     // frees the stage once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(bar_tfull + 8 * acc);   // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;                        // TMEM lane quarter this warp may access
        uint32_t acc_phase[2] = {0, 0};
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++it) {
            const int acc = it & 1;
            int b, tr, tc;
            decode_tile(p, tile, &b, &tr, &tc);
            const int jm = b;                             // the modulus table has one entry per batch entry
            const ModConsts mc = load_mod_consts(p.mods, jm);
            if (!(ok = mbar_wait(bar_tfull + 8 * acc, acc_phase[acc], abort_flag, p.dev_status, kDevTimeoutEpilogue))) break;
            acc_phase[acc] ^= 1u;
            tcgen05_fence_after();
            const int64_t row = (int64_t)tr * BM + quarter * 32 + lane;
            const int64_t col0 = (int64_t)tc * BN;
            int8_t* orow = p.out + (int64_t)b * p.out_plane_stride + row * p.ldp + col0;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(taddr + (uint32_t)(c * 32), v);
                tmem_ld_wait();
                if (row < p.R) {
#pragma unroll
                    for (int g = 0; g < 2; ++g) {            // two 16-byte groups
                        const int64_t col = col0 + c * 32 + g * 16;
                        if (col < p.ldp) {
                            uint4* dst = reinterpret_cast<uint4*>(orow + c * 32 + g * 16);
                            if (p.accumulate) reduce_store16<true>(v + g * 16, dst, mc);
                            else reduce_store16<false>(v + g * 16, dst, mc);
                        }
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);   // this warp has drained its quarter
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

cudaError_t launch_gemm_tcgen05(const GemmArgs& a, int64_t k_limit, int sm_count, cudaStream_t st, int* launches) {
    using namespace cfg;
    if (a.R <= 0 || a.Cn <= 0 || a.nbatch <= 0 || a.row_end <= a.row_begin) return cudaSuccess;
    static bool attr_set_dev[kMaxDevices] = {};
    bool& attr_set = attr_set_dev[current_device_slot()];
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(gemm_i8_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    CUtensorMap map_row, map_col;
    if (!make_plane_map(&map_row, a.rowop, a.row_planes, a.R, a.Kp, BM) || !make_plane_map(&map_col, a.colop, a.col_planes, a.Cn, a.Kp, BN))
        return cudaErrorInvalidValue;
    GemmKernelParams p;
    p.R = a.R;
    p.Cn = a.Cn;
    p.tr0 = (int)(a.row_begin / BM);
    p.tiles_r = (int)((a.row_end - a.row_begin + BM - 1) / BM);
    p.tiles_c = (int)((a.Cn + BN - 1) / BN);
    p.nbatch = a.nbatch;
    p.row_plane0 = a.row_plane0;
    p.col_plane0 = a.col_plane0;
    p.out = a.out;
    p.ldp = a.ldp;
    p.out_plane_stride = a.R * a.ldp;
    p.mods = a.mods;
    p.dev_status = a.dev_status;
    p.band = p.tiles_r < 8 ? p.tiles_r : 8;
    const int64_t total_tiles = (int64_t)p.tiles_r * p.tiles_c * p.nbatch;
    if (total_tiles > INT32_MAX) return cudaErrorInvalidValue;
    const int grid = (int)(total_tiles < sm_count ? total_tiles : sm_count);
    const int kblocks_total = (int)(a.Kp / BK);
    const int chunk = (int)((k_limit / BK) > 0 ? (k_limit / BK) : 1);   // K slices per launch that keep int32 exact
    for (int kb0 = 0; kb0 < kblocks_total; kb0 += chunk) {
        p.kblock0 = kb0;
        p.kblocks = (kblocks_total - kb0 < chunk) ? kblocks_total - kb0 : chunk;
        p.accumulate = (kb0 > 0 || a.accumulate) ? 1 : 0;
        gemm_i8_tcgen05_kernel<<<grid, THREADS, SMEM_BYTES, st>>>(map_row, map_col, p);
        ++*launches;
    }
    return cudaGetLastError();
}

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
    int64_t chunk = (k_limit / cfg::BK) * cfg::BK;
    if (chunk <= 0) chunk = cfg::BK;
    dim3 grid((unsigned)((a.Cn + 15) / 16), (unsigned)((a.row_end - a.row_begin + 15) / 16), (unsigned)a.nbatch);
    gemm_i8_check_kernel<<<grid, 256, 0, st>>>(a.rowop, a.colop, a.R, a.Cn, a.Kp, chunk, a.row_plane0, a.col_plane0, a.out, a.ldp, a.mods,
                                               a.row_begin, a.row_end, a.accumulate);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace gemm2m

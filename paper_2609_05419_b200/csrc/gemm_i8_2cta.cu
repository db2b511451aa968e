// Batched int8 GEMM with modular epilogue, Eq. (2b), on CTA pairs: tcgen05.mma.cta_group::2.
//
// Two CTAs on neighbouring SMs (a cluster of 2) share one 256 x 256 output tile.  Each CTA loads its own 128 rows of the
// row operand and its own 128-row half of the column operand (no multicast), the leader CTA issues one MMA of
// M = 256, N = 256, K = 32 per instruction that reads both CTAs' shared memory, and each CTA ends up with its 128 x 256
// half of the int32 accumulator in its own TMEM.  Per SM this needs 2/3 of the shared-memory operand traffic of a
// 128 x 256 single-CTA tile and 2/3 of the L2 -> SM traffic, which is what bounds a dense int8 contraction.
//
// Roles per CTA (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer (leader CTA only) and TMEM allocation,
// warps 2-5 = epilogue (tcgen05.ld, exact reduction mod m_j, one byte per entry to HBM).
// Barriers: the leader's full[s] collects the bytes of both CTAs' loads; the MMA's commit is multicast to both CTAs'
// empty[s] and tmem_full[a]; both CTAs' epilogue warps arrive on the leader's tmem_empty[a].
// Every wait is bounded in time.  When one gives up, a code is recorded, every role of both CTAs leaves its loop, and before
// shared memory, barriers and TMEM go away the pair makes sure nothing is still in flight: the MMA issuer commits what it has
// issued to a barrier of its own and waits for it; the leader's producer squares the byte counts of the stages that only one
// CTA had got to (both producers publish how many stage fills they issued) and waits for the last fill of every stage, which
// completes when both CTAs' copies of it have landed.  These waits are bounded too (0.1 s each).
#include "gemm_ptx.cuh"

namespace gemm2m {

namespace cfg2 {
constexpr int BM = 128;        // rows of the row operand per CTA (TMEM lanes); the pair covers 256
constexpr int BN = 256;        // rows of the column operand per pair (TMEM columns); each CTA loads 128 of them
constexpr int BK = kGemmBK;
constexpr int UMMA_K = 32;
#ifndef GEMM2M_PAIR_STAGES
#define GEMM2M_PAIR_STAGES 6
#endif
constexpr int STAGES = GEMM2M_PAIR_STAGES;
constexpr int ROW_TILE_BYTES = BM * BK;          // 16 KB
constexpr int COL_HALF_BYTES = (BN / 2) * BK;    // 16 KB
constexpr int STAGE_BYTES = ROW_TILE_BYTES + COL_HALF_BYTES;
constexpr int THREADS = 192;
constexpr int TMEM_COLS = 512;                   // two accumulators of 256 columns
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 + 256;   // tiles (1024-byte aligned) + barriers and flags
}  // namespace cfg2

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory offset in CTA `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_cluster_u32(uint32_t cluster_addr) {
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
    return v;
}
// TMA load of this CTA's tile whose completion bytes are credited to a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void umma_i8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives (once all MMAs issued so far have completed) on the barrier at this offset in every CTA of `mask`.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"(mask)
                 : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(cfg2::THREADS, 1)
gemm_i8_tcgen05_pair_kernel(const __grid_constant__ CUtensorMap map_row, const __grid_constant__ CUtensorMap map_col,
                            const __grid_constant__ GemmKernelParams p) {
    using namespace cfg2;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    unsigned char* gen_base = smem_raw + (tiles_base - raw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + (size_t)STAGES * STAGE_BYTES);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * STAGES, bar_tempty = bar_tfull + 16;
    const uint32_t bar_drain = bar_tempty + 16;           // give-up path only: the MMA issuer's last commit
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 5);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile uint32_t* fills_issued = reinterpret_cast<volatile uint32_t*>(tmem_slot + 2);   // stage fills this CTA's producer issued

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0 = leader
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(bar_tfull + 8 * a, 1); mbar_init(bar_tempty + 8 * a, 8); }   // 4 warps of each CTA
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        *fills_issued = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();                                  // the peer's barriers exist before anything signals them
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    wait_for_prior_kernels();                            // barriers and TMEM are set up; the planes are read from here on

    const int tiles_per_batch = p.tiles_r * p.tiles_c;
    const int total_tiles = tiles_per_batch * p.nbatch;
    const uint32_t peer_abort = map_to_cta(smem_u32(const_cast<int*>(abort_flag)), rank ^ 1u);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            const uint32_t leader_full = map_to_cta(bar_full, 0);
            uint32_t stage = 0, phase = 0, fills = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < total_tiles; tile += npairs) {
                int b, tr, tc;
                decode_tile(p, tile, &b, &tr, &tc);
                const int row0 = tr * (2 * BM) + (int)rank * BM;
                const int col0 = tc * BN + (int)rank * (BN / 2);
                for (int kb = 0; kb < p.kblocks; ++kb) {
                    if (!(ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, kDevTimeoutProducer, p.wait_ns))) break;
                    const uint32_t dst = tiles_base + stage * STAGE_BYTES;
                    if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * STAGE_BYTES);   // both CTAs' bytes
                    const int x = (p.kblock0 + kb) * BK;
                    tma_load_3d_pair(dst, &map_row, leader_full + 8 * stage, x, row0, p.row_plane0 + b);
                    tma_load_3d_pair(dst + ROW_TILE_BYTES, &map_col, leader_full + 8 * stage, x, col0, p.col_plane0 + b);
                    ++fills;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            *fills_issued = fills;
            if (!ok) st_cluster_u32(peer_abort, 1u);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_idesc_i8(2 * BM, BN);
            uint32_t stage = 0, phase = 0;
            uint32_t acc_phase[2] = {0, 0};
            bool ok = true;
            int it = 0;
            for (int tile = pair; ok && tile < total_tiles; tile += npairs, ++it) {
                const int acc = it & 1;
                if (!(ok = mbar_wait(bar_tempty + 8 * acc, acc_phase[acc] ^ 1u, abort_flag, p.dev_status, kDevTimeoutMma, p.wait_ns))) break;
                acc_phase[acc] ^= 1u;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < p.kblocks; ++kb) {
                    if (!(ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.dev_status, kDevTimeoutMma, p.wait_ns))) break;
                    tcgen05_fence_after();
                    const uint32_t a_addr = tiles_base + stage * STAGE_BYTES;
                    const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(a_addr + ROW_TILE_BYTES);
#pragma unroll
                    for (int k4 = 0; k4 < BK / UMMA_K; ++k4)
                        umma_i8_pair(d_tmem, adesc + (uint64_t)(k4 * (UMMA_K >> 4)), bdesc + (uint64_t)(k4 * (UMMA_K >> 4)), idesc,
                                     (uint32_t)((kb | k4) != 0));
                    umma_commit_pair(bar_empty + 8 * stage, 3);     // the stage is free in both CTAs
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit_pair(bar_tfull + 8 * acc, 3);    // accumulator complete in both CTAs
            }
            if (!ok) st_cluster_u32(peer_abort, 1u);
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
        const int quarter = warp & 3;
        const uint32_t leader_tempty = map_to_cta(bar_tempty, 0);
        uint32_t acc_phase[2] = {0, 0};
        bool ok = true;
        int it = 0;
        for (int tile = pair; ok && tile < total_tiles; tile += npairs, ++it) {
            const int acc = it & 1;
            int b, tr, tc;
            decode_tile(p, tile, &b, &tr, &tc);
            const int jm = b;                             // the modulus table has one entry per batch entry
            const ModConsts mc = load_mod_consts(p.mods, jm);
            if (!(ok = mbar_wait(bar_tfull + 8 * acc, acc_phase[acc], abort_flag, p.dev_status, kDevTimeoutEpilogue, p.wait_ns))) break;
            acc_phase[acc] ^= 1u;
            tcgen05_fence_after();
            const int64_t row = (int64_t)tr * (2 * BM) + (int64_t)rank * BM + quarter * 32 + lane;
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
                    for (int g = 0; g < 2; ++g) {
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
            if (lane == 0) {
                if (rank == 0) mbar_arrive(bar_tempty + 8 * acc);
                else mbar_arrive_cluster(leader_tempty + 8 * acc);
            }
        }
        if (!ok && lane == 0) st_cluster_u32(peer_abort, 1u);
    }

    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();            // neither CTA's shared memory, barriers or TMEM may go away while the peer still uses them
    // A role that gives up sets its CTA's flag and then the peer's, both before this point, so the two CTAs agree on the flag.
    if (*abort_flag) {
        // Bulk copies may still be on their way into either CTA's shared memory, each crediting its bytes to the leader's
        // full[stage].  The producers run at most STAGES fills apart (a fill of a stage follows the MMAs that consumed the
        // stage's previous fill, which needed both CTAs' bytes), so every barrier is short of, or ahead by, at most one fill:
        // the leader takes the missing peer bytes off, or announces the peer bytes it had not got to, and then waits for
        // the last fill of every stage to complete.
        if (warp == 1 && lane == 0 && rank == 0) {
            // MMAs already issued (by this thread, whichever role gave up) still read both CTAs' shared memory and write both
            // TMEMs: commit them to a barrier of their own and wait until they are through
            umma_commit_pair(bar_drain, 1);
            mbar_wait_quiet(bar_drain, 0, kDrainLimitNs);
        }
        if (warp == 0 && lane == 0 && rank == 0) {
            const uint32_t mine = *fills_issued, peers = ld_cluster_u32(map_to_cta(smem_u32(const_cast<uint32_t*>(fills_issued)), 1u));
            for (uint32_t f = min(mine, peers); f < max(mine, peers); ++f) {
                const uint32_t bar = bar_full + 8 * (f % STAGES);
                if (peers < mine) mbar_complete_tx(bar, STAGE_BYTES);
                else mbar_arrive_expect_tx(bar, STAGE_BYTES);
            }
            const uint32_t fills = max(mine, peers);
            for (uint32_t s = 0; s < (uint32_t)STAGES && s < fills; ++s) {
                const uint32_t last = s + STAGES * ((fills - 1 - s) / STAGES);       // last fill of stage s
                mbar_wait_quiet(bar_full + 8 * s, (last / STAGES) & 1u, kDrainLimitNs);
            }
        }
        __syncthreads();
        cluster_sync_all();
    }
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

cudaError_t launch_gemm_tcgen05_pair(const GemmArgs& a, int64_t k_limit, int sm_count, cudaStream_t st, int* launches) {
    using namespace cfg2;
    if (a.R <= 0 || a.Cn <= 0 || a.nbatch <= 0 || a.row_end <= a.row_begin) return cudaSuccess;
    static bool attr_set_dev[kMaxDevices] = {};
    bool& attr_set = attr_set_dev[current_device_slot()];
    static int max_pairs_dev[kMaxDevices] = {};
    int& max_pairs = max_pairs_dev[current_device_slot()];
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(gemm_i8_tcgen05_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
        if (err != cudaSuccess) return err;
        cudaLaunchConfig_t qc = {};
        qc.gridDim = dim3((unsigned)(sm_count & ~1), 1, 1);
        qc.blockDim = dim3(THREADS, 1, 1);
        qc.dynamicSmemBytes = SMEM_BYTES;
        cudaLaunchAttribute qa[1];
        qa[0].id = cudaLaunchAttributeClusterDimension;
        qa[0].val.clusterDim.x = 2;
        qa[0].val.clusterDim.y = 1;
        qa[0].val.clusterDim.z = 1;
        qc.attrs = qa;
        qc.numAttrs = 1;
        int clusters = 0;
        err = cudaOccupancyMaxActiveClusters(&clusters, gemm_i8_tcgen05_pair_kernel, &qc);
        if (err != cudaSuccess) return err;
        max_pairs = clusters > 0 ? clusters : sm_count / 2;
        if (max_pairs > sm_count / 2) max_pairs = sm_count / 2;
        attr_set = true;
    }
    CUtensorMap map_row, map_col;
    if (!make_plane_map(&map_row, a.rowop, a.row_planes, a.R, a.Kp, BM) || !make_plane_map(&map_col, a.colop, a.col_planes, a.Cn, a.Kp, BN / 2))
        return cudaErrorInvalidValue;
    GemmKernelParams p;
    p.R = a.R;
    p.Cn = a.Cn;
    p.tr0 = (int)(a.row_begin / (2 * BM));
    p.tiles_r = (int)((a.row_end - a.row_begin + 2 * BM - 1) / (2 * BM));
    p.tiles_c = (int)((a.Cn + BN - 1) / BN);
    p.nbatch = a.nbatch;
    p.row_plane0 = a.row_plane0;
    p.col_plane0 = a.col_plane0;
    p.out = a.out;
    p.ldp = a.ldp;
    p.out_plane_stride = a.R * a.ldp;
    p.mods = a.mods;
    p.dev_status = a.dev_status;
    p.wait_ns = kWaitLimitNs;
    p.band = p.tiles_r < 8 ? p.tiles_r : 8;
    const int64_t total_tiles = (int64_t)p.tiles_r * p.tiles_c * p.nbatch;
    if (total_tiles > INT32_MAX) return cudaErrorInvalidValue;
    const int pairs = (int)(total_tiles < max_pairs ? total_tiles : max_pairs);
    const int kblocks_total = (int)(a.Kp / BK);
    const int chunk = (int)((k_limit / BK) > 0 ? (k_limit / BK) : 1);
    for (int kb0 = 0; kb0 < kblocks_total; kb0 += chunk) {
        p.kblock0 = kb0;
        p.kblocks = (kblocks_total - kb0 < chunk) ? kblocks_total - kb0 : chunk;
        p.accumulate = (kb0 > 0 || a.accumulate) ? 1 : 0;
        cudaError_t err = launch_chained(gemm_i8_tcgen05_pair_kernel, dim3(2 * pairs), dim3(THREADS), SMEM_BYTES, st, map_row, map_col, p);   // cluster size is a kernel attribute
        if (err != cudaSuccess) return err;
        ++*launches;
    }
    return cudaGetLastError();
}

// The bounded wait of the GEMM kernel on its own: one thread, one barrier that nobody arrives on.  No pipeline, no bulk copy,
// no TMEM: the wait runs out after budget_ns, records its code and the kernel returns.
__global__ void __launch_bounds__(32) wait_selftest_kernel(int* dev_status, unsigned long long budget_ns) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(smem_u32(&bar), 0, &abort_flag, dev_status, kDevTimeoutSelfTest, budget_ns);
    }
}

cudaError_t launch_wait_selftest(int* dev_status, unsigned long long budget_ns, cudaStream_t st) {
    wait_selftest_kernel<<<1, 32, 0, st>>>(dev_status, budget_ns);
    return cudaGetLastError();
}

}  // namespace gemm2m

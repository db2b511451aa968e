// PTX wrappers and small host helpers shared by the tcgen05 int8 GEMM kernels (mbarrier, TMA, tcgen05 MMA / TMEM,
// descriptors, bounded waits).
#pragma once
#include "common.cuh"

#include <cuda.h>

namespace gemm2m {

constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s: default budget of every device-side wait (GemmKernelParams::wait_ns)
constexpr unsigned long long kDrainLimitNs = 100000000ull;   // 0.1 s: budget of the waits of the give-up path, per barrier
constexpr int kGemmBK = 128;                                  // bytes of K per pipeline stage (one 128-byte swizzle row)

// ------------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// The same, letting the hardware park the warp for up to `hint_ns` while the phase is incomplete (fewer polling instructions).
__device__ __forceinline__ bool mbar_try_wait_parked(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false (and records `code`) if the barrier did not complete within limit_ns or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* dev_status, int code,
                                          unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try_wait_parked(bar, parity, 10000u)) return true;
        if ((spins & 15u) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                atomicCAS(dev_status, kDevOk, code);
                return false;
            }
        }
    }
}

// Bounded wait of the give-up path: no status, no flag; returns whether the phase completed.
__device__ __forceinline__ bool mbar_wait_quiet(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
    const unsigned long long t0 = global_timer_ns();
    while (!mbar_try_wait_parked(bar, parity, 10000u))
        if (global_timer_ns() - t0 > limit_ns) return false;
    return true;
}
// Takes `bytes` off the pending transaction count of the barrier's current phase (bytes that were announced and will not come).
__device__ __forceinline__ void mbar_complete_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.complete_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 bytes apart, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
    d |= (uint64_t)1 << 16;                    // leading-dimension byte offset: unused for swizzled K-major
    d |= (uint64_t)(1024 >> 4) << 32;          // stride-dimension byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                    // 128-byte swizzle
    return d;
}

// Instruction descriptor for kind::i8: signed 8-bit A and B, both K-major, int32 accumulator, M x N tile.
__host__ __device__ constexpr uint32_t make_idesc_i8(int M, int N) {
    return (2u << 4)                   // D format: S32
           | (1u << 7) | (1u << 10)    // A, B format: signed 8-bit
           | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives on the mbarrier once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
          "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]),
          "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
          "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
          "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Constants of the epilogue's reduction modulo the modulus of one batch entry (see ModTable).
struct ModConsts {
    uint32_t w;        // int8 x4: sym(256^b mod m), b = 0..3
    int y0;            // bit pattern of the float Y0, minus sym(2^31 mod m)
    int neg_m;
    float inv_m, cq;
};
__device__ __forceinline__ ModConsts load_mod_consts(const ModTable& t, int b) {
    return ModConsts{t.w[b], t.y0[b], -t.m[b], t.inv_m[b], t.cq[b]};
}

// Symmetric residue of an int32 accumulator x, in the low byte of the result.  x + 2^31 (one XOR) is a non-negative 32-bit
// number whose four unsigned bytes are contracted with 256^b mod m by one dp4a; the accumulation starts at the bit pattern
// of the float Y0 minus sym(2^31 mod m) (folded into y0 by the table builder) plus `extra`, a residue to be added.  The sum
// is the bit pattern of Y0 + x' with x' = x (mod m) and |x'| small; one FMA gives 1.5 2^23 + rint(x'/m) exactly and one
// integer multiply-add leaves x' - rint(x'/m) m in the low byte (the proof is the residue kernels').  No conversions, no
// fix-ups.
__device__ __forceinline__ uint32_t sym_reduce_acc(uint32_t x, const ModConsts c, int extra) {
    int y;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(y) : "r"(x ^ 0x80000000u), "r"(c.w), "r"(c.y0 + extra));
    const int t = __float_as_int(fmaf(__int_as_float(y), c.inv_m, c.cq));
    return (uint32_t)(t * c.neg_m + y);
}

// 16 consecutive accumulators of one TMEM lane -> 16 symmetric residues packed into one 16-byte vector.
// ACC: add the residues already stored at `dst` first (later K chunks, second product of a rank-2k update).
template <bool ACC>
__device__ __forceinline__ void reduce_store16(const uint32_t* v, uint4* dst, const ModConsts c) {
    uint32_t old[4] = {0, 0, 0, 0};
    if (ACC) { const uint4 o = *dst; old[0] = o.x; old[1] = o.y; old[2] = o.z; old[3] = o.w; }
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint32_t b[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) b[e] = sym_reduce_acc(v[q * 4 + e], c, ACC ? (int)(int8_t)(old[q] >> (8 * e)) : 0);
        w[q] = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
    }
    *dst = make_uint4(w[0], w[1], w[2], w[3]);
}

struct GemmKernelParams {
    int64_t R, Cn;           // valid rows of the row operand / of the column operand
    int kblocks;             // K slices of BK bytes in this launch
    int kblock0;             // first K slice (K split)
    int tiles_r, tiles_c, nbatch;
    int row_plane0, col_plane0;
    int8_t* out;
    int64_t ldp, out_plane_stride;
    int accumulate;          // add the residues already stored in `out` (later K chunks)
    int band;                // tile rasterisation: row tiles per band (see decode_tile)
    int tr0;                 // first row tile of this launch (tiles_r counts the row tiles of the launch)
    ModTable mods;
    int* dev_status;
    unsigned long long wait_ns;   // budget of every device-side wait
};

// Linear tile index -> (batch, row tile, column tile).  Within a batch the tiles are walked in bands of `band` row tiles,
// column by column inside a band, so that the tiles in flight at any time (one per CTA or CTA pair, consecutive indices)
// cover about band x (CTAs / band) tiles and share their operand slices through L2 instead of re-reading them from HBM.
__device__ __forceinline__ void decode_tile(const GemmKernelParams& p, int tile, int* b, int* tr, int* tc) {
    const int per_batch = p.tiles_r * p.tiles_c;
    *b = tile / per_batch;
    const int rem = tile - *b * per_batch;
    const int per_band = p.band * p.tiles_c;
    const int band_idx = rem / per_band, in_band = rem - band_idx * per_band;
    const int rows_here = min(p.band, p.tiles_r - band_idx * p.band);
    *tc = in_band / rows_here;
    *tr = p.tr0 + band_idx * p.band + (in_band - *tc * rows_here);
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// planes: [P][rows][Kp] int8; box = 128 bytes of K x box_rows rows of one plane; rows beyond `rows` read as zero.
inline bool make_plane_map(CUtensorMap* map, const int8_t* base, int64_t planes, int64_t rows, int64_t Kp, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)Kp, (cuuint64_t)rows, (cuuint64_t)planes};
    const cuuint64_t strides[2] = {(cuuint64_t)Kp, (cuuint64_t)Kp * (cuuint64_t)rows};
    const cuuint32_t box[3] = {(cuuint32_t)kGemmBK, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


}  // namespace gemm2m

// Steps 3 + 4 (Eq. 2a) with the byte-weight contraction on the tensor cores: a selectable variant of residues_fp_kernel
// (gemm2m_debug_set_residue_kernel), bit-identical planes.  It is not the default: on a 4096 x 4096 operand with 16 moduli it
// takes 302 us against 215 us for the dp4a kernel, because the synchronisation between its three roles and the per-value
// epilogue cost more instructions than the dp4a chains they replace.
//
// The residue of a quantised part x modulo m is the dot product of the balanced base-256 digits of x with the weights
// 256^b mod m (Section 3.1 applied to the digits).  For every residue plane p (X+ and X- of a 2M modulus, X_r, X_i and
// X_r + X_i of a 3M modulus) that is one row of weights over the 2 x 12 digit positions of an element, so all planes of
// all elements are one small int8 matrix product
//     D[plane, element] = sum_pos W[plane, pos] * digit[element, pos],
// which tcgen05.mma.kind::i8 forms with the planes along M (TMEM lanes) and the elements along N (TMEM columns).  A thread
// of the epilogue then owns one plane and reads consecutive elements of it: the modulus is a per-thread constant and the
// reduction is one add, one FP32 FMA and one integer multiply-add per residue.  The weight rows are repeated in every lane
// quarter (every half when there are more than 32 planes), so one instruction of shape M = 128, N = 128 gives each of
// the four epilogue warps the sums of all 128 elements of a step and each warp reduces its own share of the columns.
// The bytes go to a shared-memory buffer and leave as full 128-byte lines with the lanes of a warp along one plane: a store
// with one plane per lane touches 32 pages 16 to 64 MiB apart per instruction and ran five times slower.
//
// One CTA = 416 threads, 256 TMEM columns (two accumulator buffers), two CTAs per SM; a tile is 8 operand rows x 128 k,
// consumed in 8 steps of 128 elements.
#include "gemm_ptx.cuh"

#include <cstring>

namespace gemm2m {

namespace rtc {
constexpr int ROWS = 8, KT = 128, THREADS = 416;   // 8 reducing warps, 4 quantising warps, 1 issuing warp
constexpr int RING = 4;                         // tiles of raw elements in flight per CTA
constexpr int STEP = 128;                       // elements per MMA step = TMEM columns per accumulator buffer
constexpr int TMEM_COLS = 256;                  // two accumulator buffers
constexpr int DIGIT_BYTES = STEP * 32;          // 32 digit positions per element
constexpr int OUT_STRIDE = 144;                 // bytes per lane in the output staging buffer: 128 + 16 spreads the banks
constexpr int IMAGE_ROWS_MAX = 128;             // weight image: the plane rows, repeated for every lane quarter (or half)
constexpr size_t MIN_SMEM = 76 * 1024;          // keeps the residency at two CTAs per SM: 2 x 256 TMEM columns
}  // namespace rtc

// Per-plane constants of the tensor-core residue kernel.
struct alignas(16) TcPlaneTable {
    int8_t w[kMaxPlanes][32];      // positions 0..11: weights of the real part's digits, 16..27: of the imaginary part's
    int32_t y0[kMaxPlanes];        // bit pattern of the float Y0 of the plane's modulus (see ResidueTable::magic)
    float inv_m[kMaxPlanes], cq[kMaxPlanes];
    int32_t neg_m[kMaxPlanes];
    int nplanes;
};

static void build_tc_plane_table(const ResidueTable& r, TcPlaneTable* t) {
    std::memset(t, 0, sizeof(*t));
    const int n2 = r.n2, n3 = r.nmod - r.n2;
    t->nplanes = 2 * n2 + 3 * n3;
    auto unpack = [](uint32_t lo, uint32_t hi, uint32_t top, int8_t* out) {
        for (int b = 0; b < 4; ++b) {
            out[b] = (int8_t)(lo >> (8 * b));
            out[4 + b] = (int8_t)(hi >> (8 * b));
            out[8 + b] = (int8_t)(top >> (8 * b));
        }
    };
    auto fill = [&](int p, int j, int re_sign, int im_sign, bool im_plain) {
        int8_t w[12], ws[12];
        unpack(r.w_lo[j], r.w_hi[j], r.w_top[j], w);
        if (im_plain) std::memcpy(ws, w, 12);
        else unpack(r.ws_lo[j], r.ws_hi[j], r.ws_top[j], ws);
        for (int b = 0; b < 12; ++b) {
            t->w[p][b] = (int8_t)(re_sign * w[b]);
            t->w[p][16 + b] = (int8_t)(im_sign * ws[b]);
        }
        t->y0[p] = r.magic[j];
        t->inv_m[p] = r.inv_m[j];
        t->cq[p] = r.cq[j];
        t->neg_m[p] = -r.m[j];
    };
    for (int j = 0; j < n2; ++j) {
        fill(j, j, 1, 1, false);            // X+ = X_r + s X_i
        fill(n2 + j, j, 1, -1, false);      // X- = X_r - s X_i
    }
    for (int j3 = 0; j3 < n3; ++j3) {
        const int j = n2 + j3;
        fill(2 * n2 + j3, j, 1, 0, true);              // X_r
        fill(2 * n2 + n3 + j3, j, 0, 1, true);         // X_i
        fill(2 * n2 + 2 * n3 + j3, j, 1, 1, true);     // X_r + X_i
    }
}

// K-major operand without swizzle: 8 rows x 16 bytes form a contiguous 128-byte core matrix; the two core matrices that
// make up K = 32 bytes are 128 bytes apart, 8-row groups 256 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc_plain(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(128 >> 4) << 16;           // leading-dimension byte offset: next core matrix along K
    d |= (uint64_t)(256 >> 4) << 32;           // stride-dimension byte offset: next 8-row group
    d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
    return d;                                  // swizzle field 0: none
}

template <typename T> struct RtcRaw;
template <> struct RtcRaw<double> { using type = double2; };
template <> struct RtcRaw<float> { using type = float2; };

template <int BYTES>
__device__ __forceinline__ void rtc_cp_async_zfill(void* smem_dst, const void* gmem_src, bool valid) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const int src_bytes = valid ? BYTES : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;" ::"r"(d), "l"(gmem_src), "n"(BYTES), "r"(src_bytes) : "memory");
}

// Balanced base-256 digits of a two's complement value: adding 128 to every byte (with carries) and flipping the top bit
// of every byte leaves bytes that, read as signed, satisfy x = sum_b digit_b 256^b.
__device__ __forceinline__ uint4 balanced_digits(long long x) {
    const unsigned long long k = 0x8080808080808080ull;
    const unsigned long long rec = ((unsigned long long)x + k) ^ k;
    return make_uint4((uint32_t)rec, (uint32_t)(rec >> 32), 0u, 0u);
}
__device__ __forceinline__ uint4 balanced_digits_wide(__int128 x) {   // |x| < 2^94
    const unsigned __int128 k = ((unsigned __int128)0x80808080ull << 64) | 0x8080808080808080ull;
    const unsigned __int128 rec = ((unsigned __int128)x + k) ^ k;
    return make_uint4((uint32_t)rec, (uint32_t)(rec >> 32), (uint32_t)(rec >> 64), 0u);
}

template <typename T> struct RtcBits;
template <> struct RtcBits<double> {
    static constexpr int kMantBits = 52, kBias = 1023;
    __device__ static unsigned long long mag(double v) { return (unsigned long long)__double_as_longlong(v) & 0x7FFFFFFFFFFFFFFFull; }
    __device__ static bool neg(double v) { return __double_as_longlong(v) < 0; }
};
template <> struct RtcBits<float> {
    static constexpr int kMantBits = 23, kBias = 127;
    __device__ static unsigned long long mag(float v) { return (unsigned long long)((uint32_t)__float_as_int(v) & 0x7FFFFFFFu); }
    __device__ static bool neg(float v) { return __float_as_int(v) < 0; }
};

// trunc(v 2^-e) for a finite v from its bit pattern, as a 128-bit integer (|result| < 2^92 by the scaling rule).
template <typename T>
__device__ __forceinline__ __int128 quantise_bits(T v, int e) {
    using F = RtcBits<T>;
    const unsigned long long mag = F::mag(v);
    const int E = (int)(mag >> F::kMantBits);
    unsigned long long mant = mag & ((1ull << F::kMantBits) - 1);
    if (E) mant |= (1ull << F::kMantBits);
    const int sh = max(E, 1) - (F::kBias + F::kMantBits) - e;      // v = mant 2^(max(E,1) - bias - mantbits)
    unsigned __int128 q;
    if (sh >= 0) q = (unsigned __int128)mant << min(sh, 74);        // the clamp only keeps the shift defined
    else q = (-sh > 63) ? 0 : (mant >> (-sh));
    return F::neg(v) ? -(__int128)q : (__int128)q;
}

// Bounded wait for a barrier that completes within microseconds: plain polling, no parking.
__device__ __forceinline__ bool mbar_wait_short(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* dev_status, int code) {
    unsigned long long t0 = 0;
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spins & 255u) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                atomicCAS(dev_status, kDevOk, code);
                return false;
            }
        }
    }
}

// Roles: warps 0-7 reduce and store (warps w and w + 4 read TMEM lanes 32 w ..), warps 8-11 quantise (one element per thread and
// step, fetched by the same thread with cp.async into slots nobody else reads, so no block-wide barrier is needed),
// warp 12 allocates TMEM and issues the MMAs.  Digits and accumulators are double buffered; four mbarrier pairs hand them
// round: digits_full (4 quantising warps) -> MMA -> digits_empty and tmem_full (tcgen05.commit) -> reduce ->
// tmem_empty (8 warps).  The quantising warps never store to global memory, so the proxy fence after their shared-memory
// writes does not wait for anything slow.
template <typename T, bool WIDE, int NB>
__global__ void __launch_bounds__(rtc::THREADS, 2)
residues_tc_kernel(const T* __restrict__ X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K, int64_t Kp,
                   const int32_t* __restrict__ e, const __grid_constant__ TcPlaneTable tab, int8_t* __restrict__ planes,
                   int* dev_status) {
    using namespace rtc;
    using Raw = typename RtcRaw<T>::type;
    constexpr int RPB = 128 / NB;      // weight rows (TMEM lanes) per element block
    constexpr int CPB = STEP / NB;     // elements (TMEM columns) per block
    constexpr int STEPS = ROWS * KT / STEP;   // 8 steps per tile
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* digits = smem_raw;                                  // 2 x [16 groups][2 K halves][8 rows][16 B]
    unsigned char* image = smem_raw + 2 * DIGIT_BYTES;                 // [16 groups][2][8][16 B]
    uint64_t* bars = reinterpret_cast<uint64_t*>(image + IMAGE_ROWS_MAX * 32);
    const uint32_t bar_dfull = smem_u32(bars), bar_dempty = bar_dfull + 16, bar_tfull = bar_dfull + 32, bar_tempty = bar_dfull + 48;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    unsigned char* outbuf = image + IMAGE_ROWS_MAX * 32 + 128;              // [128 TMEM lanes][OUT_STRIDE]: residue bytes of one row group
    Raw* ring = reinterpret_cast<Raw*>(outbuf + 128 * OUT_STRIDE);           // [RING][STEPS][128 threads]

    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;

    if (t == 0) {
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_dfull + 8 * a, 4);
            mbar_init(bar_dempty + 8 * a, 1);
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, 8);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 12) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // weight image, 128 rows: every block of RPB rows (TMEM lanes) holds the planes once more, so that one MMA gives every
    // lane quarter the sums of all elements of the step and each warp can take its own share of the columns
    for (int idx = t; idx < 128 * 2; idx += THREADS) {
        const int row = idx >> 1, half = idx & 1;
        const int p = row % RPB;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (p < tab.nplanes) v = *reinterpret_cast<const uint4*>(&tab.w[p][16 * half]);
        *reinterpret_cast<uint4*>(image + (row >> 3) * 256 + half * 128 + (row & 7) * 16) = v;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int64_t ktiles = Kp / KT;
    const int64_t total = ((R + ROWS - 1) / ROWS) * ktiles;
    bool ok = true;

    if (warp < 8) {
        // ------------------------------------------------------------------ reduce + store: one TMEM lane = one plane of one block;
        // warps w and w + 4 share lane quarter w and take one half each of the block's columns
        const int quarter = warp & 3, half = warp >> 2;
        constexpr int CW = CPB / 2;                                // columns per warp and step
        const int my_lane = 32 * quarter + lane;
        const int my_block = my_lane / RPB, my_plane = my_lane % RPB;
        const bool plane_ok = my_plane < tab.nplanes;
        const int pp = plane_ok ? my_plane : 0;
        const int y0 = tab.y0[pp], neg_m = tab.neg_m[pp];
        const float inv_m = tab.inv_m[pp], cq = tab.cq[pp];
        const uint32_t taddr = tmem_base + ((uint32_t)(32 * quarter) << 16) + (uint32_t)(my_block * CPB + half * CW);
        unsigned char* my_out = outbuf + my_lane * OUT_STRIDE + half * CW;
        const int64_t plane_stride = R * Kp;
        uint32_t g = 0;
        for (int64_t tile = blockIdx.x; ok && tile < total; tile += gridDim.x) {
            const int64_t row0 = (tile / ktiles) * ROWS, k0 = (tile % ktiles) * KT;
#pragma unroll 1
            for (int step = 0; step < STEPS; ++step, ++g) {
                const uint32_t buf = g & 1u, ph = (g >> 1) & 1u;
                if (!(ok = mbar_wait_short(bar_tfull + 8 * buf, ph, abort_flag, dev_status, kDevTimeoutEpilogue))) break;
                tcgen05_fence_after();
                const int rg = step / NB, kb = step % NB;
                uint32_t v[CW];
                if constexpr (CW == 16) tmem_ld16(taddr + buf * STEP, v);
                else tmem_ld32(taddr + buf * STEP, v);
                tmem_ld_wait();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);      // the accumulators are in registers: the MMA may go on
#pragma unroll
                for (int c = 0; c < CW / 16; ++c) {
                    uint32_t w[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t b4[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int y = (int)v[16 * c + 4 * q + i] + y0;                          // bits of the float Y0 + x
                            const int tq = __float_as_int(fmaf(__int_as_float(y), inv_m, cq));      // bits of 1.5 2^23 + rint(x/m)
                            b4[i] = (uint32_t)(tq * neg_m + y);                                     // low byte: x - rint(x/m) m
                        }
                        w[q] = __byte_perm(__byte_perm(b4[0], b4[1], 0x0040), __byte_perm(b4[2], b4[3], 0x0040), 0x5410);
                    }
                    *reinterpret_cast<uint4*>(my_out + CPB * kb + 16 * c) = make_uint4(w[0], w[1], w[2], w[3]);
                }
                if (kb == NB - 1) {
                    // The 128 k of this row group are complete for every plane: write them out with the lanes of a warp along
                    // the bytes of a plane (full 128-byte lines, one or two planes per instruction) instead of one plane per lane.
                    asm volatile("bar.sync 1, 256;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int run = j * 32 + (t >> 3);                  // plane-major: run = plane * NB + block
                        const int p = run / NB, b = run % NB;
                        const int64_t orow = row0 + NB * rg + b;
                        if (p < tab.nplanes && orow < R) {
                            const uint4 val = *reinterpret_cast<const uint4*>(outbuf + (b * RPB + p) * OUT_STRIDE + 16 * (t & 7));
                            *reinterpret_cast<uint4*>(planes + (int64_t)p * plane_stride + orow * Kp + k0 + 16 * (t & 7)) = val;
                        }
                    }
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                }
            }
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------------ quantise: thread-private ring of raw elements
        const int pt = t - 256;                                  // 0..127
        // element of this thread within a step: block (= operand row within the step) and k within the block.
        // Consecutive threads take consecutive k when k is contiguous in memory, consecutive rows otherwise.
        const int el_block = k_contiguous ? pt / CPB : pt % NB;
        const int el_k = k_contiguous ? pt % CPB : pt / NB;
        const int el = el_block * CPB + el_k;                    // row of the digit matrix = TMEM column
        unsigned char* my_digits = digits + (el >> 3) * 256 + (el & 7) * 16;
        Raw* my_ring = ring + pt;
        auto issue = [&](int64_t tile, int slot) {
            if (tile < total) {
                const int64_t row0 = (tile / ktiles) * ROWS, k0 = (tile % ktiles) * KT;
#pragma unroll
                for (int step = 0; step < STEPS; ++step) {
                    const int64_t row = row0 + NB * (step / NB) + el_block, k = k0 + CPB * (step % NB) + el_k;
                    const bool in = row < R && k < K;
                    const T* src = in ? (k_contiguous ? X + 2 * (k + row * ld) : X + 2 * (row + k * ld)) : X;
                    rtc_cp_async_zfill<sizeof(Raw)>(my_ring + (slot * STEPS + step) * 128, src, in);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        int64_t tile = blockIdx.x;
#pragma unroll
        for (int s = 0; s < RING - 1; ++s) issue(tile + (int64_t)s * gridDim.x, s);
        uint32_t g = 0;
        for (int it = 0; ok && tile < total; tile += gridDim.x, ++it) {
            issue(tile + (int64_t)(RING - 1) * gridDim.x, (it + RING - 1) % RING);
            asm volatile("cp.async.wait_group %0;" ::"n"(RING - 1) : "memory");
            const int64_t row0 = (tile / ktiles) * ROWS;
            const Raw* src = my_ring + (it % RING) * STEPS * 128;
#pragma unroll 1
            for (int step = 0; step < STEPS; ++step, ++g) {
                const uint32_t buf = g & 1u, ph = (g >> 1) & 1u;
                const int64_t row = row0 + NB * (step / NB) + el_block;
                uint4 dr = make_uint4(0, 0, 0, 0), di = dr;
                if (row < R) {
                    const int ex = __ldg(e + row);
                    Raw v = src[step * 128];
                    if (conj) v.y = -v.y;                     // conjugated operand
                    if (ex != kExpNonFinite) {
                        if (!WIDE && ex > -1000 && ex < 1000) {
                            // x 2^-e is an exact FP64 product (or underflows towards zero, where the truncation is zero
                            // anyway) and its truncation to int64 is one conversion; |x 2^-e| < 2^62 by the scaling rule
                            const double scale = __longlong_as_double((long long)(1023 - ex) << 52);
                            dr = balanced_digits(__double2ll_rz((double)v.x * scale));
                            di = balanced_digits(__double2ll_rz((double)v.y * scale));
                        } else if (!WIDE) {
                            dr = balanced_digits((long long)quantise_bits<T>(v.x, ex));
                            di = balanced_digits((long long)quantise_bits<T>(v.y, ex));
                        } else {
                            dr = balanced_digits_wide(quantise_bits<T>(v.x, ex));
                            di = balanced_digits_wide(quantise_bits<T>(v.y, ex));
                        }
                    }
                }
                if (!(ok = mbar_wait_short(bar_dempty + 8 * buf, ph ^ 1u, abort_flag, dev_status, kDevTimeoutProducer))) break;
                *reinterpret_cast<uint4*>(my_digits + buf * DIGIT_BYTES) = dr;
                *reinterpret_cast<uint4*>(my_digits + buf * DIGIT_BYTES + 128) = di;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_dfull + 8 * buf);      // one arrival per warp: 128 arrivals on one barrier serialise
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else if (lane == 0) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc = make_idesc_i8(128, STEP);
        uint32_t g = 0;
        for (int64_t tile = blockIdx.x; ok && tile < total; tile += gridDim.x) {
#pragma unroll 1
            for (int step = 0; step < STEPS; ++step, ++g) {
                const uint32_t buf = g & 1u, ph = (g >> 1) & 1u;
                if (!(ok = mbar_wait_short(bar_dfull + 8 * buf, ph, abort_flag, dev_status, kDevTimeoutMma))) break;
                if (!(ok = mbar_wait_short(bar_tempty + 8 * buf, ph ^ 1u, abort_flag, dev_status, kDevTimeoutMma))) break;
                tcgen05_fence_after();
                umma_i8(tmem_base + buf * STEP, make_smem_desc_plain(smem_u32(image)),
                        make_smem_desc_plain(smem_u32(digits) + buf * DIGIT_BYTES), idesc, 0u);
                umma_commit(bar_dempty + 8 * buf);     // the digits have been read
                umma_commit(bar_tfull + 8 * buf);      // the accumulators are complete
            }
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    if (warp == 12) {
        __syncwarp();
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <typename T>
cudaError_t launch_residues_tc(const T* X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K, int64_t Kp, const int32_t* e,
                               const ResidueTable& rtab, bool wide, int8_t* planes, int* dev_status, int sm_count, cudaStream_t st,
                               int* launches) {
    using namespace rtc;
    if (R <= 0 || Kp <= 0) return cudaSuccess;
    TcPlaneTable tab;
    build_tc_plane_table(rtab, &tab);
    size_t smem = (size_t)2 * DIGIT_BYTES + IMAGE_ROWS_MAX * 32 + 128 + 128 * OUT_STRIDE + (size_t)RING * ROWS * KT * 2 * sizeof(T);
    if (smem < MIN_SMEM) smem = MIN_SMEM;
    const int64_t total = ((R + ROWS - 1) / ROWS) * (Kp / KT);
    const int64_t resident = (int64_t)(sm_count > 0 ? sm_count : 148) * 2;
    const unsigned grid = (unsigned)(total < resident ? total : resident);
    auto go = [&](auto kernel) -> cudaError_t {
        cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        kernel<<<grid, THREADS, smem, st>>>(X, ld, k_contiguous, conj, R, K, Kp, e, tab, planes, dev_status);
        return cudaGetLastError();
    };
    cudaError_t err;
    if (tab.nplanes <= 32) err = wide ? go(residues_tc_kernel<T, true, 4>) : go(residues_tc_kernel<T, false, 4>);
    else err = wide ? go(residues_tc_kernel<T, true, 2>) : go(residues_tc_kernel<T, false, 2>);
    ++*launches;
    return err;
}

template cudaError_t launch_residues_tc<double>(const double*, int64_t, bool, bool, int64_t, int64_t, int64_t, const int32_t*, const ResidueTable&,
                                                bool, int8_t*, int*, int, cudaStream_t, int*);
template cudaError_t launch_residues_tc<float>(const float*, int64_t, bool, bool, int64_t, int64_t, int64_t, const int32_t*, const ResidueTable&,
                                               bool, int8_t*, int*, int, cudaStream_t, int*);

}  // namespace gemm2m

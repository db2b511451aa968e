// Algorithm 1 steps 4-7 for the rank-k family (Section 5): only C+ = A+ A-^T was computed; C- = C+^T, so entry (i, j) of the
// result takes c+ = C+[i, j] and c- = C+[j, i] of every modulus.  cp: [nmod][n][ldp] int8 with cp[jm][col][row] = C+_jm[row, col].
// The sums over the planes are the same 8-bit tensor-core contraction as for the complex GEMMs (post_fp.cu), with the planes read
// twice: directly (contiguous along i) and mirrored (contiguous along j).  Lower triangle only; on the diagonal c- = c+, the
// imaginary part's weights cancel modulo M and the imaginary part is exactly zero.
#include "post_mma.cuh"

namespace gemm2m {

constexpr int kHkI = 64, kHkJ = 16;              // tile: 64 rows i x 16 columns j of C
constexpr int kHkWarps = 4, kHkThreads = 32 * kHkWarps;
constexpr int kHkDirStride = kHkJ * (kHkI / 4) + 8;   // words per directly read plane: [jj][16 words of i], + 8 (32 banks for a warp's loads)
constexpr int kHkMirStride = kHkI * (kHkJ / 4) + 4;   // words per mirrored plane: [ii][4 words of j], + 4

__host__ __device__ constexpr int hk_block_words(int halves, int nb) {   // halves: 16-plane halves of K per kind (direct / mirrored)
    return 16 * halves * (kHkDirStride + kHkMirStride) + kHkWarps * 32 * pf_row_words(nb);
}

// 4 x 4 byte transpose: out[c] byte r = in[r] byte c.
__device__ __forceinline__ void transpose4(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, uint32_t (&o)[4]) {
    const uint32_t lo01 = __byte_perm(w0, w1, 0x5140), hi01 = __byte_perm(w0, w1, 0x7362);
    const uint32_t lo23 = __byte_perm(w2, w3, 0x5140), hi23 = __byte_perm(w2, w3, 0x7362);
    o[0] = __byte_perm(lo01, lo23, 0x5410);
    o[1] = __byte_perm(lo01, lo23, 0x7632);
    o[2] = __byte_perm(hi01, hi23, 0x5410);
    o[3] = __byte_perm(hi01, hi23, 0x7632);
}

// A block handles a 64 x 16 tile of the lower triangle.  Both views of the planes are pulled into shared memory with
// asynchronous 16-byte copies: direct [plane][jj][64 bytes along i] and mirrored [plane][ii][16 bytes along j].  A warp takes
// 32 consecutive i x 4 consecutive j at a time; lane (g, t) owns the 4 x 4 block i = 4g .. 4g+3, j = 4 jq .. 4 jq + 3 of it.  For
// every j of the block the four i are one word of a direct plane; for every i the four j are one word of a mirrored plane, so a
// 4 x 4 byte transpose of the mirrored words gives, per j, the same "four neighbouring i" word as the direct view.  From there
// on a group (32 i, one j) is processed as in post_fp.cu: bytes to [0, 255], plane-by-element transpose, MMAs against the digit
// matrix, chunks through shared memory, finish per element, coalesced store along i.
// HV: 16-plane halves of K per view (1 for up to 16 moduli, 2 beyond).  REAL_OUT: C is real (SYRK / SYR2K), only X_r is formed.
template <int HV, int NB, bool REAL_OUT>
__global__ void __launch_bounds__(kHkThreads) post_herk_kernel(const int8_t* __restrict__ cp, int64_t ldp, int64_t n, int64_t i_begin, int nmod,
                                                               const int32_t* __restrict__ eA, const uint32_t* __restrict__ frags,
                                                               const __grid_constant__ PostConsts pc, double* __restrict__ C, int64_t ldc) {
    extern __shared__ __align__(16) uint32_t hk_smem[];
    wait_for_prior_kernels();
    constexpr int KS = HV;                                   // K-steps of 32 slots: HV halves direct + HV halves mirrored
    constexpr int kRow = pf_row_words(NB);
    uint32_t* sdir = hk_smem;
    uint32_t* smir = hk_smem + 16 * HV * kHkDirStride;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    uint32_t* xch = smir + 16 * HV * kHkMirStride + warp * 32 * kRow;
    const int64_t ibase = i_begin + (int64_t)blockIdx.x * kHkI, jbase = (int64_t)blockIdx.y * kHkJ;
    if (ibase + kHkI - 1 < jbase) return;                    // tile entirely above the diagonal
    const int64_t plane = n * ldp;
    // direct view: for each modulus and column j of the tile, 64 bytes along i (4 copies)
    for (int idx = threadIdx.x; idx < nmod * kHkJ * (kHkI / 16); idx += kHkThreads) {
        const int v = idx & 3, jj = (idx >> 2) & (kHkJ - 1), jm = idx / (kHkJ * 4);
        const int64_t i = ibase + 16 * v, j = jbase + jj;
        if (j < n && i < ldp) cp_async16(sdir + jm * kHkDirStride + jj * (kHkI / 4) + 4 * v, cp + (int64_t)jm * plane + j * ldp + i);
    }
    // mirrored view: for each modulus and row i of the tile, the 16 bytes C+[jbase .. jbase+15, i]
    for (int idx = threadIdx.x; idx < nmod * kHkI; idx += kHkThreads) {
        const int ii = idx & (kHkI - 1), jm = idx / kHkI;
        const int64_t i = ibase + ii;
        if (i < n && jbase < ldp) cp_async16(smir + jm * kHkMirStride + ii * (kHkJ / 4), cp + (int64_t)jm * plane + i * ldp + jbase);
    }
    cp_async_commit_group();

    // K slots: [direct planes, padded to 16 HV][mirrored planes, padded to 16 HV]; K-step s, half h is slot group 2s + h
    uint32_t bf[KS][NB][2];
#pragma unroll
    for (int s = 0; s < KS; ++s)
#pragma unroll
        for (int q = 0; q < NB; ++q) {
            bf[s][q][0] = __ldg(frags + ((s * NB + q) * 2 + 0) * 32 + lane);
            bf[s][q][1] = __ldg(frags + ((s * NB + q) * 2 + 1) * 32 + lane);
        }
    uint32_t chunk_hi[NB / 2];
#pragma unroll
    for (int c = 0; c < NB / 2; ++c) chunk_hi[c] = 0x43380000u + ((uint32_t)(32 * ((t & 1) * (NB / 2) + c)) << 20);
    uint32_t two16;
    asm("mov.b32 %0, 65536;" : "=r"(two16));
    cp_async_wait_pending<0>();
    __syncthreads();

    constexpr int kBlocks = (kHkI / 32) * (kHkJ / 4);        // 32 x 4 blocks of the tile: 8, two per warp
#pragma unroll 1
    for (int blk = warp; blk < kBlocks; blk += kHkWarps) {
        const int i32 = 32 * (blk & (kHkI / 32 - 1)), jq = blk / (kHkI / 32);
        if (ibase + i32 + 31 < jbase + 4 * jq) continue;     // block entirely above the diagonal
        // mirrored words of this lane's four i, transposed to one word per j: mir[half][r][jo] = bytes (i = 4g .. 4g+3) of plane t + 4r, j = 4 jq + jo
        uint32_t mir[HV][4][4];
#pragma unroll
        for (int h = 0; h < HV; ++h)
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const uint32_t* p = smir + (16 * h + t + 4 * r) * kHkMirStride + (i32 + 4 * g) * (kHkJ / 4) + jq;
                transpose4(p[0], p[kHkJ / 4], p[2 * (kHkJ / 4)], p[3 * (kHkJ / 4)], mir[h][r]);
            }
        const int ei_lane = ibase + i32 + lane < n ? __ldg(eA + ibase + i32 + lane) : 0;
#pragma unroll 1
        for (int jo = 0; jo < 4; ++jo) {
            const int64_t j = jbase + 4 * jq + jo;
            int acc[2][NB][4];
#pragma unroll
            for (int s = 0; s < KS; ++s) {
                uint32_t a0[4], a1[4];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int slot_half = 2 * s + h;         // halves 0 .. HV-1 are direct planes, HV .. 2 HV - 1 mirrored
                    uint32_t w[4];
                    if (slot_half < HV) {
                        const uint32_t* p = sdir + (16 * slot_half + t) * kHkDirStride + (4 * jq + jo) * (kHkI / 4) + i32 / 4 + g;
#pragma unroll
                        for (int r = 0; r < 4; ++r) w[r] = p[4 * r * kHkDirStride];
                    } else {
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const uint32_t(&m4)[4] = mir[slot_half >= HV ? slot_half - HV : 0][r];
                            w[r] = jo == 0 ? m4[0] : jo == 1 ? m4[1] : jo == 2 ? m4[2] : m4[3];
                        }
                    }
                    uint32_t el[4];
                    transpose4(w[0] ^ 0x80808080u, w[1] ^ 0x80808080u, w[2] ^ 0x80808080u, w[3] ^ 0x80808080u, el);   // residue + 128
                    a0[2 * h] = el[0];
                    a0[2 * h + 1] = el[1];
                    a1[2 * h] = el[2];
                    a1[2 * h + 1] = el[3];
                }
#pragma unroll
                for (int q = 0; q < NB; ++q) {
                    if (s == 0) {
                        mma_u8(acc[0][q], a0, bf[s][q][0], bf[s][q][1]);
                        mma_u8(acc[1][q], a1, bf[s][q][0], bf[s][q][1]);
                    } else {
                        mma_u8_acc(acc[0][q], a0, bf[s][q][0], bf[s][q][1]);
                        mma_u8_acc(acc[1][q], a1, bf[s][q][0], bf[s][q][1]);
                    }
                }
            }
            __syncwarp();                                   // the previous group's reads of the exchange buffer are done
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                unsigned long long chunk[NB / 2];
#pragma unroll
                for (int c = 0; c < NB / 2; ++c) {
                    const uint32_t a = (uint32_t)(acc[e >> 1][2 * c][2 * (e & 1)] + 256 * acc[e >> 1][2 * c][2 * (e & 1) + 1]);
                    const uint32_t b = (uint32_t)(acc[e >> 1][2 * c + 1][2 * (e & 1)] + 256 * acc[e >> 1][2 * c + 1][2 * (e & 1) + 1]);
                    chunk[c] = pack_chunk(a, b, chunk_hi[c], two16);
                }
                uint32_t* row = xch + (4 * g + e) * kRow + t * NB;
                if constexpr (NB % 4 == 0) {
#pragma unroll
                    for (int c = 0; c < NB / 2; c += 2) *reinterpret_cast<ulonglong2*>(row + 2 * c) = make_ulonglong2(chunk[c], chunk[c + 1]);
                } else {
#pragma unroll
                    for (int c = 0; c < NB / 2; ++c) *reinterpret_cast<unsigned long long*>(row + 2 * c) = chunk[c];
                }
            }
            __syncwarp();
            double br[NB], bi[NB];
            {
                const double2* row = reinterpret_cast<const double2*>(xch + lane * kRow);
#pragma unroll
                for (int c = 0; c < NB / 2; ++c) {
                    const double2 vr = row[c], vi = row[NB / 2 + c];
                    br[2 * c] = vr.x; br[2 * c + 1] = vr.y;
                    bi[2 * c] = vi.x; bi[2 * c + 1] = vi.y;
                }
            }
            const int64_t i = ibase + i32 + lane;
            const int ej = j < n ? __ldg(eA + j) : 0;
            double hr, lr, re, im = 0.0;
            crt_finish32<NB>(br, pc.off[0], pc, &hr, &lr);
            const int e = (int)((uint32_t)ei_lane + (uint32_t)ej);
            const bool fast = e > -1000 && e < 1000;        // 2^e is a normal number: one multiplication
            re = fast ? (NB == 2 ? hr : hr + lr) * __longlong_as_double((long long)(e + 1023) << 52) : scale_pow2(NB == 2 ? hr : hr + lr, e);
            if (!REAL_OUT) {
                double hi, li;
                crt_finish32<NB>(bi, pc.off[1], pc, &hi, &li);
                im = fast ? (NB == 2 ? hi : hi + li) * __longlong_as_double((long long)(e + 1023) << 52) : scale_pow2(NB == 2 ? hi : hi + li, e);
            }
            if (ei_lane == kExpNonFinite || ej == kExpNonFinite) re = im = __longlong_as_double(0x7FF8000000000000ll);
            if (i < n && j < n && i >= j) {
                if (REAL_OUT) C[i + j * ldc] = re;
                else *reinterpret_cast<double2*>(C + 2 * (i + j * ldc)) = make_double2(re, im);
            }
        }
    }
}

template <int HV, int NB, bool REAL_OUT>
static cudaError_t launch_post_herk_v(const int8_t* cp, int64_t ldp, int64_t n, int64_t i_begin, int64_t i_end, int nmod, const int32_t* eA,
                                      const PostMmaTable& tab, const uint32_t* dev_frags, double* C, int64_t ldc, cudaStream_t st) {
    constexpr size_t smem = (size_t)hk_block_words(HV, NB) * sizeof(uint32_t);
    static bool attr_set_dev[kMaxDevices] = {};
    bool& attr_set = attr_set_dev[current_device_slot()];
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(post_herk_kernel<HV, NB, REAL_OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    const int64_t tiles_j = (i_end + kHkJ - 1) / kHkJ;     // lower triangle: columns up to the last row of the range
    if (tiles_j > 65535) return cudaErrorInvalidValue;     // n beyond 65535 * 16 columns: far beyond any workspace
    dim3 grid((unsigned)((i_end - i_begin + kHkI - 1) / kHkI), (unsigned)tiles_j);
    launch_chained(post_herk_kernel<HV, NB, REAL_OUT>, grid, dim3(kHkThreads), smem, st, cp, ldp, n, i_begin, nmod, eA, dev_frags, tab.c, C, ldc);
    return cudaGetLastError();
}

cudaError_t launch_post_herk(const int8_t* cp, int64_t ldp, int64_t n, int64_t i_begin, int64_t i_end, const int32_t* eA, const PostMmaTable& tab,
                             const uint32_t* dev_frags, double* C, int64_t ldc, bool real_out, cudaStream_t st, int* launches) {
    if (n <= 0 || i_end <= i_begin) return cudaSuccess;
    const int hv = tab.c.planes / 32;                      // 16-slot halves per view
    cudaError_t err = cudaErrorInvalidValue;
#define GEMM2M_HERK_CASE(HV, NB)                                                                                                        \
    if (hv == HV && tab.c.nb == NB)                                                                                                      \
        err = real_out ? launch_post_herk_v<HV, NB, true>(cp, ldp, n, i_begin, i_end, tab.nmod, eA, tab, dev_frags, C, ldc, st)          \
                       : launch_post_herk_v<HV, NB, false>(cp, ldp, n, i_begin, i_end, tab.nmod, eA, tab, dev_frags, C, ldc, st);
    GEMM2M_HERK_CASE(1, 2) GEMM2M_HERK_CASE(1, 4) GEMM2M_HERK_CASE(2, 4) GEMM2M_HERK_CASE(2, 6)
#undef GEMM2M_HERK_CASE
    if (err == cudaSuccess) ++*launches;
    return err;
}

}  // namespace gemm2m

// Algorithm 1 steps 4 (Eq. 2c; Eq. 1 for the 3M moduli of the hybrid), 5, 6, 7 for the complex GEMMs: from the residue planes of
// the products to C.  Per output element the work is X = sum over planes of (residue) x (folded CRT weight) mod M for the real
// and the imaginary part, an exact integer of up to 184 bits.  The weights (reduced to [0, M)) are written in base-256 digits,
// which turns the sums over the planes into a small 8-bit contraction, [elements x planes] . [planes x digit columns], that
// runs on the tensor cores (warp-level m16n8k32 MMAs, int32 accumulators; residues moved to [0, 255] so that every column
// sum is non-negative, at most 56 . 255 . 255 < 2^22).  What is left per element is to add the digit columns up (integer, then
// FP64 on 32-bit-spaced chunks), remove the multiple of M, round once and scale by 2^(e_i + f_j).
// Bound by HBM traffic: 1 byte per plane read, 16 (8) bytes written per element.
#include "post_mma.cuh"

namespace gemm2m {

#ifndef GEMM2M_POST_WARPS
#define GEMM2M_POST_WARPS 4
#endif
#ifndef GEMM2M_POST_GROUPS
#define GEMM2M_POST_GROUPS 4
#endif
constexpr int kPfWarps = GEMM2M_POST_WARPS;     // warps per block
constexpr int kPfGroups = GEMM2M_POST_GROUPS;   // MMA groups of 32 elements per warp and step
constexpr int kPfThreads = 32 * kPfWarps;
constexpr int kPfSpan = 32 * kPfGroups * kPfWarps;      // consecutive row indices i per step of a block
constexpr int kPfStrideW = kPfSpan / 4 + 4;     // words per staged plane: + 4, so that the 16-byte rows of 8 consecutive planes cover the 32 banks
#ifndef GEMM2M_POST_STAGES
#define GEMM2M_POST_STAGES 2
#endif
constexpr int kPfStages = GEMM2M_POST_STAGES;   // staging ring: the next step is on its way while this one is processed (3 stages of 512 rows,
                                                // 3 or 4 stages of 256 rows: 5-14 % slower at 8192^3)
constexpr int kPfIlp = 1;                       // groups of a warp whose elements are finished together (one exchange buffer each);
                                                // 2 and 4 measured 5 and 15 % slower at 8192^3 (fewer blocks fit), also with the
                                                // finishes written out step by step across the groups
static_assert(kPfGroups % kPfIlp == 0, "whole batches of groups");
static_assert(kPfSpan % 128 == 0, "plane stride = 4 mod 32 words");

__host__ __device__ constexpr int pf_block_words(int kh, int nb) { return kPfStages * 16 * kh * kPfStrideW + kPfWarps * kPfIlp * 32 * pf_row_words(nb); }

// cpm: [planes][n][ldp] int8 (row index i contiguous); plane = n ldp is the plane stride; ncols columns starting at the
// pointers given.  The work is cut into steps of kPfSpan consecutive i of one column j, numbered column by column within a
// block of rows; every thread block takes an equal, contiguous share of the steps.  The planes x kPfSpan residue bytes of a step
// are pulled into shared memory with asynchronous 16-byte copies while the previous step is processed.  A warp owns 32 kPfGroups
// of the i; for each group of 32 it loads the MMA operand (rows = elements, K = planes) with the transposing 8-bit matrix load
// (a staged plane's 16 consecutive element bytes are one row of the matrix in shared memory; the load hands lane (g, t) the
// bytes of planes 4t..4t+3 for elements g and g + 8, which is the operand fragment), moves the bytes to [0, 255],
// multiplies by the digit matrix held in registers, packs each run of four digit-column sums into one 64-bit chunk,
// and passes the chunks through shared memory so that every lane ends up with all chunks of one element, which it finishes and
// stores (the 32 lanes of a warp cover 32 consecutive i).  Many warps per SM matter more here than long steps: the per-element finish is a
// chain of dependent FP64 operations.
// KH: 16-plane halves of K that are staged and contracted (1, 2 or 4).
template <typename T, int KH, int NB, bool AXPBY>
__global__ void __launch_bounds__(kPfThreads) post_fp_kernel(const int8_t* __restrict__ cpm, int64_t ldp, int64_t m, int64_t plane, int ncols,
                                                             const int32_t* __restrict__ eA, const int32_t* __restrict__ eB,
                                                             const uint32_t* __restrict__ frags, const __grid_constant__ PostConsts pc,
                                                             T* __restrict__ C, int64_t ldc, const PostScalars sc) {
    static_assert(NB % 2 == 0, "whole chunks per lane");
    extern __shared__ __align__(16) uint32_t pf_smem[];
    wait_for_prior_kernels();
    constexpr int KS = (KH + 1) / 2, kHalves = KH == 1 ? 1 : 2;     // K-steps of 32 planes; halves of a step in use
    constexpr int kStageWords = 16 * KH * kPfStrideW;
    constexpr int kRow = pf_row_words(NB);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    // The element of a group that this lane finishes: exchange row `lane` = 4 g' + e' holds row g' (e' odd: g' + 8) of the 16-element
    // tile e' / 2 (a row order in which the 16-byte stores of the chunks and the 16-byte loads of the rows are both free of bank conflicts)
    const int el = 16 * ((lane >> 1) & 1) + 8 * (lane & 1) + (lane >> 2);
    uint32_t* xch = pf_smem + kPfStages * kStageWords + warp * kPfIlp * 32 * kRow;
    const int64_t total = ((m + kPfSpan - 1) / kPfSpan) * ncols;
    int64_t step = total * blockIdx.x / gridDim.x;
    const int64_t step_end = total * (blockIdx.x + 1) / gridDim.x;
    if (step >= step_end) return;
    int ibk = (int)(step / ncols), j = (int)(step - (int64_t)ibk * ncols);
    const int planes = pc.planes;

    constexpr int kVecs = kPfSpan / 16;                         // 16-byte vectors per plane and step
    const int sv = threadIdx.x % kVecs, sp = threadIdx.x / kVecs;   // staging: this thread copies vector sv of the planes sp, sp + kPfThreads / kVecs, ...
    auto issue = [&](int ibk_, int j_, int stage) {
        const int64_t ib = (int64_t)ibk_ * kPfSpan;
        if (16 * sv + 16 <= ldp - ib) {                         // ldp is a multiple of 16: whole vectors up to the padded end of the column
            const int8_t* src = cpm + (int64_t)j_ * ldp + ib + 16 * sv + (int64_t)sp * plane;
            uint32_t* dst = pf_smem + stage * kStageWords + sp * kPfStrideW + 4 * sv;
            for (int p = sp; p < planes; p += kPfThreads / kVecs) {
                cp_async16(dst, src);
                src += (kPfThreads / kVecs) * plane;
                dst += (kPfThreads / kVecs) * kPfStrideW;
            }
        }
        cp_async_commit_group();
    };
    // the ring is filled kPfStages - 1 steps ahead: (pibk, pj) is the step the next copy is for
    int pibk = ibk, pj = j;
    int64_t pstep = step;
#pragma unroll
    for (int a = 0; a < kPfStages - 1; ++a) {
        if (pstep < step_end) issue(pibk, pj, a);
        else cp_async_commit_group();
        ++pstep;
        if (++pj == ncols) { pj = 0; ++pibk; }
    }

    uint32_t bf[KS][NB][2];
#pragma unroll
    for (int s = 0; s < KS; ++s)
#pragma unroll
        for (int q = 0; q < NB; ++q) {
            bf[s][q][0] = __ldg(frags + ((s * NB + q) * 2 + 0) * 32 + lane);
            bf[s][q][1] = kHalves > 1 ? __ldg(frags + ((s * NB + q) * 2 + 1) * 32 + lane) : 0u;
        }
    // High word of chunk c of this lane: 1.5 2^52 with the weight 2^(32k) of the chunk, k = (t & 1) NB/2 + c, in its exponent.
    uint32_t chunk_hi[NB / 2];
#pragma unroll
    for (int c = 0; c < NB / 2; ++c) chunk_hi[c] = 0x43380000u + ((uint32_t)(32 * ((t & 1) * (NB / 2) + c)) << 20);
    int ea[kPfGroups] = {}, ea_block = -1;
    uint32_t two16;
    asm("mov.b32 %0, 65536;" : "=r"(two16));

    for (int n = 0; step < step_end; ++step, ++n) {
        int jn = j + 1, ibkn = ibk;
        if (jn == ncols) { jn = 0; ++ibkn; }
        if (pstep < step_end) issue(pibk, pj, (n + kPfStages - 1) % kPfStages);
        else cp_async_commit_group();                       // an empty group keeps the count of pending groups uniform
        ++pstep;
        if (++pj == ncols) { pj = 0; ++pibk; }
        cp_async_wait_pending<kPfStages - 1>();
        __syncthreads();
        const uint32_t* st = pf_smem + (n % kPfStages) * kStageWords;
        const int64_t ib = (int64_t)ibk * kPfSpan + 32 * kPfGroups * warp;    // first row of this warp
        if (ibk != ea_block) {
#pragma unroll
            for (int it = 0; it < kPfGroups; ++it) ea[it] = ib + 32 * it + el < m ? __ldg(eA + ib + 32 * it + el) : 0;
            ea_block = ibk;
        }
        const int fb = __ldg(eB + j);
        T* dst0 = C + 2 * (ib + el + (int64_t)j * ldc);       // this lane's element of the warp's first group
        const int64_t rows_left = m - ib - el;               // group `it` is inside the matrix for this lane if 32 it < rows_left
        // MMA phase of group `it`: operand gather, contraction, chunks into the exchange buffer xb
        auto contract = [&](int it, uint32_t* xb) {
            int acc[2][NB][4];
            // rows of the staged planes holding this group's 32 elements: lane L addresses plane L of the K-step (16 bytes = elements 0..15)
            const uint32_t rows = (uint32_t)__cvta_generic_to_shared(st) + (kHalves > 1 ? lane : (lane & 15)) * (4 * kPfStrideW) + 32 * (kPfGroups * warp + it);
#pragma unroll
            for (int s = 0; s < KS; ++s) {
                uint32_t a0[4], a1[4];                      // A operands of the two 16-row tiles: elements 0..15 and 16..31 of the group
                if (kHalves > 1) {
                    load_a_k32(a0, rows + s * (32 * 4 * kPfStrideW));
                    load_a_k32(a1, rows + s * (32 * 4 * kPfStrideW) + 16);
                } else {
                    uint32_t x0[2], x1[2];
                    load_a_k16(x0, rows);
                    load_a_k16(x1, rows + 16);
                    a0[0] = x0[0]; a0[1] = x0[1]; a1[0] = x1[0]; a1[1] = x1[1];
                    a0[2] = a0[3] = a1[2] = a1[3] = 0u;
                }
#pragma unroll
                for (int r = 0; r < 2 * kHalves; ++r) { a0[r] ^= 0x80808080u; a1[r] ^= 0x80808080u; }      // residue + 128
#pragma unroll
                for (int q = 0; q < NB; ++q) {
                    if (KH == 1) {
                        mma_u8_k16(acc[0][q], a0[0], a0[1], bf[s][q][0]);
                        mma_u8_k16(acc[1][q], a1[0], a1[1], bf[s][q][0]);
                    } else if (s == 0) {
                        mma_u8(acc[0][q], a0, bf[s][q][0], bf[s][q][1]);
                        mma_u8(acc[1][q], a1, bf[s][q][0], bf[s][q][1]);
                    } else {
                        mma_u8_acc(acc[0][q], a0, bf[s][q][0], bf[s][q][1]);
                        mma_u8_acc(acc[1][q], a1, bf[s][q][0], bf[s][q][1]);
                    }
                }
            }
            // accumulator registers 0, 1 hold row g (element g of the tile), columns 2t, 2t+1 (two neighbouring digits); registers 2, 3 the same for row g + 8
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                unsigned long long chunk[NB / 2];
#pragma unroll
                for (int c = 0; c < NB / 2; ++c) {
                    const uint32_t a = (uint32_t)(acc[e >> 1][2 * c][2 * (e & 1)] + 256 * acc[e >> 1][2 * c][2 * (e & 1) + 1]);
                    const uint32_t b = (uint32_t)(acc[e >> 1][2 * c + 1][2 * (e & 1)] + 256 * acc[e >> 1][2 * c + 1][2 * (e & 1) + 1]);
                    chunk[c] = pack_chunk(a, b, chunk_hi[c], two16);           // bits of (1.5 2^52 + a + 2^16 b) 2^(32k)
                }
                uint32_t* row = xb + (4 * g + e) * kRow + t * NB;     // tile e / 2, row g or g + 8 of it: finished by lane 4 g + e
                if constexpr (NB % 4 == 0) {
#pragma unroll
                    for (int c = 0; c < NB / 2; c += 2) *reinterpret_cast<ulonglong2*>(row + 2 * c) = make_ulonglong2(chunk[c], chunk[c + 1]);
                } else {
#pragma unroll
                    for (int c = 0; c < NB / 2; ++c) *reinterpret_cast<unsigned long long*>(row + 2 * c) = chunk[c];
                }
            }
        };
        // kPfIlp groups at a time: their contractions first, then the FP64 finishes of all of them
#pragma unroll
        for (int ip = 0; ip < kPfGroups; ip += kPfIlp) {
            __syncwarp();                                   // the previous groups' reads of the exchange buffers are done
#pragma unroll
            for (int u = 0; u < kPfIlp; ++u) contract(ip + u, xch + u * 32 * kRow);
            __syncwarp();
            double br[kPfIlp][NB], bi[kPfIlp][NB];          // lanes 0, 1 of a quad wrote the real part's chunks, lanes 2, 3 the imaginary part's
#pragma unroll
            for (int u = 0; u < kPfIlp; ++u) {
                const double2* row = reinterpret_cast<const double2*>(xch + u * 32 * kRow + lane * kRow);
#pragma unroll
                for (int c = 0; c < NB / 2; ++c) {
                    const double2 vr = row[c], vi = row[NB / 2 + c];
                    br[u][2 * c] = vr.x; br[u][2 * c + 1] = vr.y;
                    bi[u][2 * c] = vi.x; bi[u][2 * c + 1] = vi.y;
                }
            }
            double xr[kPfIlp], xi[kPfIlp];                  // lanes beyond m work on whatever the staging buffer holds; nothing of it is stored
#pragma unroll
            for (int u = 0; u < kPfIlp; ++u) {
                double hr, lr, hi, li;
                crt_finish32<NB>(br[u], pc.off[0], pc, &hr, &lr);
                crt_finish32<NB>(bi[u], pc.off[1], pc, &hi, &li);
                if (pc.im_hi != 0.0) {                       // Eisenstein variant: V sqrt(3)/2 as a double-double product, rounded once below
                    const double p = hi * pc.im_hi;
                    li = fma(hi, pc.im_lo, fma(li, pc.im_hi, fma(hi, pc.im_hi, -p)));
                    hi = p;
                }
                xr[u] = NB == 2 ? hr : hr + lr;              // the one rounding of the lifted integers
                xi[u] = hi + li;
            }
#pragma unroll
            for (int u = 0; u < kPfIlp; ++u) {
                const int it = ip + u;
                double re, im;
                const int eai = ea[it];
                const int e = (int)((uint32_t)eai + (uint32_t)fb);
                const bool bad = eai == kExpNonFinite || fb == kExpNonFinite;     // an Inf or NaN in the row of A or the column of B
                if (bad || (unsigned)(e + 999) < 1999u) {
                    // 2^e is a normal number: one multiplication by a factor built from its exponent (a NaN for a bad row / column)
                    re = xr[u] * __hiloint2double(bad ? 0x7FF80000 : (e + pc.re_shift + 1023) << 20, 0);
                    im = xi[u] * __hiloint2double(bad ? 0x7FF80000 : (e + 1023) << 20, 0);
                } else {
                    re = scale_pow2(xr[u], e + pc.re_shift);
                    im = scale_pow2(xi[u], e);
                }
                T* dst = dst0 + 64 * it;
                if (AXPBY) {
                    double yr = fma(sc.ar, re, -sc.ai * im), yi = fma(sc.ar, im, sc.ai * re);
                    if (32 * it < rows_left && (sc.br != 0.0 || sc.bi != 0.0)) {
                        const double cr = (double)dst[0], ci = (double)dst[1];
                        yr += fma(sc.br, cr, -sc.bi * ci);
                        yi += fma(sc.br, ci, sc.bi * cr);
                    }
                    re = yr;
                    im = yi;
                }
                if (32 * it < rows_left) store_cplx<T>(dst, re, im);
            }
        }
        __syncthreads();                                    // every warp is done with this stage before it is refilled
        ibk = ibkn;
        j = jn;
    }
}

// The B-operand registers of the contraction, written once per call into the workspace (the kernels read them with
// coalesced loads; as a kernel argument every lane would read a different word of the constant bank).
__global__ void __launch_bounds__(256) post_operands_kernel(const __grid_constant__ PostMmaTable tab, uint32_t* __restrict__ dst) {
    for (int i = threadIdx.x; i < kPostFragWords; i += blockDim.x) dst[i] = tab.bfrag[i];
}

cudaError_t launch_post_operands(const PostMmaTable& tab, uint32_t* dev_frags, cudaStream_t st, int* launches) {
    post_operands_kernel<<<1, 256, 0, st>>>(tab, dev_frags);
    ++*launches;
    return cudaGetLastError();
}

template <typename T, int KH, int NB, bool AXPBY>
static cudaError_t launch_post_fp_v(const int8_t* cpm, int64_t ldp, int64_t m, int64_t n, int64_t j_begin, int64_t j_end, const int32_t* eA,
                                    const int32_t* eB, const PostMmaTable& tab, const uint32_t* dev_frags, T* C, int64_t ldc,
                                    const PostScalars& sc, cudaStream_t st, int* launches) {
    constexpr size_t smem = (size_t)pf_block_words(KH, NB) * sizeof(uint32_t);
    static int resident_dev[kMaxDevices] = {};          // thread blocks the device holds at once (0 = not asked yet)
    int& resident = resident_dev[current_device_slot()];
    if (!resident) {
        cudaError_t err = cudaFuncSetAttribute(post_fp_kernel<T, KH, NB, AXPBY>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        int per_sm = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, post_fp_kernel<T, KH, NB, AXPBY>, kPfThreads, smem);
        if (err != cudaSuccess) return err;
        resident = (per_sm > 0 ? per_sm : 1) * cached_sm_count();
    }
    constexpr int64_t kColsPerLaunch = 1 << 20;           // keeps step count times warp count of a launch far inside 63 bits
    for (int64_t j0 = j_begin; j0 < j_end; j0 += kColsPerLaunch) {
        const int64_t nj = (j_end - j0 < kColsPerLaunch) ? j_end - j0 : kColsPerLaunch;
        const int64_t steps = ((m + kPfSpan - 1) / kPfSpan) * nj;
        const unsigned grid = (unsigned)(steps < resident ? steps : resident);
        launch_chained(post_fp_kernel<T, KH, NB, AXPBY>, dim3(grid), dim3(kPfThreads), smem, st, cpm + j0 * ldp, ldp, m, n * ldp, (int)nj, eA, eB + j0, dev_frags, tab.c,
                                                                        C + 2 * j0 * ldc, ldc, sc);
        ++*launches;
    }
    return cudaGetLastError();
}

template <typename T, bool AXPBY>
static cudaError_t launch_post_fp_t(const int8_t* cpm, int64_t ldp, int64_t m, int64_t n, int64_t j_begin, int64_t j_end, const int32_t* eA,
                                    const int32_t* eB, const PostMmaTable& tab, const uint32_t* dev_frags, T* C, int64_t ldc,
                                    const PostScalars& sc, cudaStream_t st, int* launches) {
    const int kh = tab.c.planes <= 16 ? 1 : 2 * tab.c.ks;           // 16-plane halves of K in use
#define GEMM2M_POST_CASE(KH, NB)                                                                                                     \
    if (kh == KH && tab.c.nb == NB)                                                                                                   \
        return launch_post_fp_v<T, KH, NB, AXPBY>(cpm, ldp, m, n, j_begin, j_end, eA, eB, tab, dev_frags, C, ldc, sc, st, launches);
    GEMM2M_POST_CASE(1, 2) GEMM2M_POST_CASE(2, 4) GEMM2M_POST_CASE(4, 4) GEMM2M_POST_CASE(4, 6)
#undef GEMM2M_POST_CASE
    return cudaErrorInvalidValue;
}

template <typename T>
cudaError_t launch_post_fp(const int8_t* cpm, int64_t ldp, int64_t m, int64_t n, int64_t j_begin, int64_t j_end, const int32_t* eA,
                           const int32_t* eB, const PostMmaTable& tab, const uint32_t* dev_frags, T* C, int64_t ldc, const double* alpha,
                           const double* beta, cudaStream_t st, int* launches) {
    if (m <= 0 || j_end <= j_begin) return cudaSuccess;
    PostScalars sc{1.0, 0.0, 0.0, 0.0};
    if (alpha) { sc.ar = alpha[0]; sc.ai = alpha[1]; }
    if (beta) { sc.br = beta[0]; sc.bi = beta[1]; }
    const bool plain = sc.ar == 1.0 && sc.ai == 0.0 && sc.br == 0.0 && sc.bi == 0.0;
    if (plain) return launch_post_fp_t<T, false>(cpm, ldp, m, n, j_begin, j_end, eA, eB, tab, dev_frags, C, ldc, sc, st, launches);
    return launch_post_fp_t<T, true>(cpm, ldp, m, n, j_begin, j_end, eA, eB, tab, dev_frags, C, ldc, sc, st, launches);
}

template cudaError_t launch_post_fp<double>(const int8_t*, int64_t, int64_t, int64_t, int64_t, int64_t, const int32_t*, const int32_t*, const PostMmaTable&, const uint32_t*, double*, int64_t, const double*, const double*, cudaStream_t, int*);
template cudaError_t launch_post_fp<float>(const int8_t*, int64_t, int64_t, int64_t, int64_t, int64_t, const int32_t*, const int32_t*, const PostMmaTable&, const uint32_t*, float*, int64_t, const double*, const double*, cudaStream_t, int*);

}  // namespace gemm2m

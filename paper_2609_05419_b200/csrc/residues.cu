// Algorithm 1 steps 3 + 4 (Eq. 2a; Eq. 1 for the 3M moduli of the hybrid; Section 3.1 for real inputs): quantisation and
// residue planes.  Bound by integer / FP32 arithmetic throughput rather than by HBM bandwidth.
#include "residues_common.cuh"

namespace gemm2m {

// =====================================================================================================
// Steps 3 + 4 (Eq. 2a): quantise by truncation and emit the symmetric int8 residues A+ / A- for every
// modulus, K contiguous.  Tiles of operand rows x 128 k are staged in shared memory (coalesced global
// reads in either orientation), then each thread owns a run of consecutive k of one row and writes
// vectors into every plane.
// =====================================================================================================
struct QPair { long long re, im; };   // quantised parts, two's complement

// Wide mode: |result| < 2^92 (19 or more moduli; 2^76 without the hybrid's 3M moduli); returned as the low 32 bits and the
// signed upper 64 bits of the 96-bit two's complement value.
template <typename T>
__device__ __forceinline__ void quantise_part_wide(T v, int e, uint32_t* lo, long long* upper) {
    using F = FpBits<T>;
    const unsigned long long mag = F::mag(v);
    const int E = (int)(mag >> F::kMantBits);
    unsigned long long mant = mag & ((1ull << F::kMantBits) - 1);
    if (E) mant |= (1ull << F::kMantBits);
    const int sh = max(E, 1) - (F::kBias + F::kMantBits) - e;
    const bool neg = (sizeof(T) == 8) ? (__double_as_longlong((double)v) < 0) : (__float_as_int((float)v) < 0);
    unsigned __int128 q;
    if (sh >= 0) q = (unsigned __int128)mant << min(sh, 74);   // a legitimate shift stays below 92 - 23; the clamp only keeps the shift defined
    else q = (-sh > 63) ? 0 : (mant >> (-sh));
    const __int128 sq = neg ? -(__int128)q : (__int128)q;
    *lo = (uint32_t)(unsigned __int128)sq;
    *upper = (long long)(sq >> 32);
}

// Eisenstein variant (Sections 3.2, 4): the lattice point (u + v sqrt(-3))/2, u = v (mod 2), nearest to (x + iy) 2^-e.
// X = |x| 2^-e and t = |y| 2^-e (2/sqrt 3) are formed as fixed-point numbers with 32 fraction bits (floor; the factor as
// the 128-bit constant floor(2^127 2/sqrt 3), the product exact in 192 bits before the shift).  The nearest point with
// u, v even is (2 rn(X), 2 rn(t/2)); it is at least as near as the nearest point with u, v odd, (2 floor(X) + 1,
// 2 floor(t/2) + 1), exactly when |X - rn(X)| + (3/2) |t - 2 rn(t/2)| <= 1.  The signs of x and y carry over to u and v.
// |u|, |v| < 2^82 by the scaling rule (below 2^62 in the narrow mode).
__device__ __forceinline__ void quantise_hex(double x, double y, int e, __int128* su_out, __int128* sv_out) {
    using F = FpBits<double>;
    typedef unsigned __int128 u128;
    auto split = [](double v, int e, unsigned long long* mant, int* sh) {
        const unsigned long long mag = F::mag(v);
        const int E = (int)(mag >> F::kMantBits);
        *mant = mag & ((1ull << F::kMantBits) - 1);
        if (E) *mant |= (1ull << F::kMantBits);
        *sh = max(E, 1) - (F::kBias + F::kMantBits) - e + 32;      // |v| 2^(32 - e) = mant 2^sh
    };
    unsigned long long mx, my;
    int shx, shy;
    split(x, e, &mx, &shx);
    split(y, e, &my, &shy);
    u128 Xf;
    if (shx >= 0) Xf = (u128)mx << min(shx, 74);                     // a legitimate shift is below 60; the clamp keeps it defined
    else Xf = (-shx > 63) ? 0 : (mx >> (-shx));
    constexpr unsigned long long kK3hi = 0x93CD3A2C8198E269ull, kK3lo = 0x0C7C0F257D92BE83ull;   // floor(2^127 2/sqrt 3)
    const u128 p0 = (u128)my * kK3lo, p1 = (u128)my * kK3hi;
    const u128 top = p1 + (p0 >> 64);                                // bits 64.. of the 181-bit product
    const int r = 127 - shy - 64;                                    // t 2^32 = product >> (127 - shy), and 127 - shy >= 64
    const u128 Tf = r >= 128 ? 0 : (r <= 0 ? top : (top >> r));
    const uint32_t fx = (uint32_t)Xf;
    const unsigned long long ft = (unsigned long long)Tf & 0x1FFFFFFFFull;
    const unsigned long long dx0 = fx < 0x80000000u ? fx : 0x100000000ull - fx;
    const unsigned long long dt0 = ft < 0x100000000ull ? ft : 0x200000000ull - ft;
    u128 u, v;
    if (2 * dx0 + 3 * dt0 <= 0x200000000ull) {
        u = ((Xf + 0x80000000ull) >> 32) << 1;
        v = ((Tf + 0x100000000ull) >> 33) << 1;
    } else {
        u = ((Xf >> 32) << 1) | 1;
        v = ((Tf >> 33) << 1) | 1;
    }
    *su_out = __double_as_longlong(x) < 0 ? -(__int128)u : (__int128)u;
    *sv_out = __double_as_longlong(y) < 0 ? -(__int128)v : (__int128)v;
}

__device__ __forceinline__ int dp4a_us(uint32_t a_unsigned, uint32_t b_signed, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a_unsigned), "r"(b_signed), "r"(c));
    return d;
}
__device__ __forceinline__ int dp4a_ss(uint32_t a_signed, uint32_t b_signed, int c) {
    int d;
    asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a_signed), "r"(b_signed), "r"(c));
    return d;
}

// Symmetric residues of the pair of sums x+ = Rv + Iv and x- = Rv - Iv, returned in the low bytes of bp / bm (two's
// complement).  The caller starts the dp4a chain at the bit pattern of the float Y0 = a multiple of 256 m in [2^23, 2^24),
// so the integers yp = bits(Y0) + x+ and ym = bits(Y0) + x- are the bit patterns of the floats Y0 + x.  One FMA with the
// constant cq = 1.5 2^23 - Y0/m gives t = 1.5 2^23 + rint(x/m) exactly (the table builder proves that the error of inv_m
// stays below the distance of x/m from a rounding boundary), and bits(y) - bits(t) m has the low byte of x - rint(x/m) m
// because the bit patterns of Y0 and of 1.5 2^23 are multiples of 256.  Per residue: one FP32 FMA, one integer multiply-add.
__device__ __forceinline__ void sym_reduce_pm(int yp, int ym, int neg_m, float inv_m, float cq, uint32_t* bp, uint32_t* bm) {
    const int tp = __float_as_int(fmaf(__int_as_float(yp), inv_m, cq));
    const int tm = __float_as_int(fmaf(__int_as_float(ym), inv_m, cq));
    *bp = (uint32_t)(tp * neg_m + yp);
    *bm = (uint32_t)(tm * neg_m + ym);
}

struct Digits { uint32_t lo, hi; };   // 4 unsigned low bytes; 4 balanced (signed) high digits
__device__ __forceinline__ Digits split_digits(long long x) {
    Digits d;
    d.lo = (uint32_t)(unsigned long long)x;
    const uint32_t hi = (uint32_t)((unsigned long long)x >> 32);
    d.hi = (hi + 0x80808080u) ^ 0x80808080u;   // hi = sum (byte_b - 128) 256^b  after adding 128 to every byte
    return d;
}
// The same for a 96-bit value given as low word and signed upper 64 bits: 8 balanced digits above the low word.
__device__ __forceinline__ Digits split_digits_wide(uint32_t lo, long long upper, uint32_t* top) {
    const unsigned long long rec = ((unsigned long long)upper + 0x8080808080808080ull) ^ 0x8080808080808080ull;
    Digits d;
    d.lo = lo;
    d.hi = (uint32_t)rec;
    *top = (uint32_t)(rec >> 32);
    return d;
}

// One symmetric residue from y = bits(Y0) + x (see sym_reduce_pm).
__device__ __forceinline__ uint32_t sym_reduce_one(int y, int neg_m, float inv_m, float cq) {
    const int t = __float_as_int(fmaf(__int_as_float(y), inv_m, cq));
    return (uint32_t)(t * neg_m + y);
}

__device__ __forceinline__ uint32_t pack4(const uint32_t (&b)[4]) {   // low bytes of four words -> one word
    return __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
}

template <int NE>
__device__ __forceinline__ void store_run(int8_t* dst, const uint32_t (&w)[NE / 4]) {
    if (NE == 16) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2 % (NE / 4)], w[3 % (NE / 4)]);
    else *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
}

// One 2M modulus (index j) of emit_run: X+ into plane j, X- into plane n2 + j.
template <int NE, bool WIDE, bool NARROW>
__device__ __forceinline__ void emit_2m(int j, int n2, const Digits (&dr)[NE], const Digits (&di)[NE], const uint32_t* tr, const uint32_t* ti,
                                        const ResidueTable& tab, int8_t* dst, int64_t plane_stride) {
    const int neg_m = -tab.m[j], y0 = tab.magic[j];
    const float inv_m = tab.inv_m[j], cq = tab.cq[j];
    const uint32_t wl = tab.w_lo[j], wh = tab.w_hi[j], sl = tab.ws_lo[j], sh = tab.ws_hi[j];
    const uint32_t wt = WIDE ? tab.w_top[j] : 0u, st = WIDE ? tab.ws_top[j] : 0u;
    // Narrow mode: every part fits 32 bits and arrives as u = x + 2^31 (four unsigned bytes): one dp4a per part, and the 2^31 comes
    // off again as 128 times the weight of byte 3 (of the real part's weights at the start of the chain, of the imaginary part's
    // weights, which carry the factor s, where the chain continues).
    const int y0n = NARROW ? y0 - 128 * (int)(int8_t)(wl >> 24) : y0;
    const int kin = NARROW ? 128 * (int)(int8_t)(sl >> 24) : 0;
    uint32_t pw[NE / 4], mw[NE / 4];
#pragma unroll
    for (int w = 0; w < NE / 4; ++w) {
        uint32_t bp[4], bm[4];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int i = 4 * w + b;
            int Ry = NARROW ? dp4a_us(dr[i].lo, wl, y0n) : dp4a_ss(dr[i].hi, wh, dp4a_us(dr[i].lo, wl, y0));  // A_r mod m (unreduced) on top of the bits of Y0
            if (WIDE) Ry = dp4a_ss(tr[i], wt, Ry);                      // digits 8..11 of the 96-bit value
            // The imaginary part's weights continue the same chain: no separate addition for the "+" sum of Eq. (2a),
            // and the "-" sum is 2 Ry - yp, a three-input integer add that does not compete with the dp4a's for their pipe.
            int yp = NARROW ? dp4a_us(di[i].lo, sl, Ry - kin) : dp4a_ss(di[i].hi, sh, dp4a_us(di[i].lo, sl, Ry));
            if (WIDE) yp = dp4a_ss(ti[i], st, yp);
            const int ym = (int)(2u * (uint32_t)Ry - (uint32_t)yp);     // the doubled bit pattern wraps, the difference does not
            sym_reduce_pm(yp, ym, neg_m, inv_m, cq, &bp[b], &bm[b]);
        }
        pw[w] = pack4(bp);
        mw[w] = pack4(bm);
    }
    store_run<NE>(dst + (int64_t)j * plane_stride, pw);
    store_run<NE>(dst + (int64_t)(n2 + j) * plane_stride, mw);
}

// Residues of NE consecutive elements of one operand row for every modulus, written as NE-byte vectors into the planes of
// that modulus: X+ and X- (Eq. 2a) for the 2M moduli, then X_r, X_i and X_r + X_i (Eq. 1 after the reduction) for the 3M
// moduli of the hybrid.  dst points at plane 0, this row, first k of the run; tr / ti (wide mode) hold the four top digits
// of each part.  NMOD > 0: exactly NMOD moduli, all of them 2M moduli, known at compile time: the loop is unrolled and the
// per-modulus constants become constant-bank operands instead of loads.
template <int NE, bool WIDE, int NMOD, bool NARROW>
__device__ __forceinline__ void emit_run(const Digits (&dr)[NE], const Digits (&di)[NE], const uint32_t* tr, const uint32_t* ti,
                                         const ResidueTable& tab, int8_t* dst, int64_t plane_stride) {
    static_assert(NE == 8 || NE == 16, "runs of 8 or 16 elements");
    if constexpr (NMOD > 0) {
#pragma unroll
        for (int j = 0; j < NMOD; ++j) emit_2m<NE, WIDE, NARROW>(j, NMOD, dr, di, tr, ti, tab, dst, plane_stride);
        return;
    }
    const int nmod = tab.nmod, n2 = tab.n2;
#pragma unroll 1
    for (int j = 0; j < n2; ++j) emit_2m<NE, WIDE, NARROW>(j, n2, dr, di, tr, ti, tab, dst, plane_stride);
    const int n3 = nmod - n2;
    int8_t* dst3 = dst + (int64_t)(2 * n2) * plane_stride;
#pragma unroll 1
    for (int j3 = 0; j3 < n3; ++j3) {
        const int j = n2 + j3;
        const int neg_m = -tab.m[j], y0 = tab.magic[j];
        const float inv_m = tab.inv_m[j], cq = tab.cq[j];
        const uint32_t wl = tab.w_lo[j], wh = tab.w_hi[j], wt = WIDE ? tab.w_top[j] : 0u;
        uint32_t rw[NE / 4], iw[NE / 4], sw[NE / 4];
#pragma unroll
        for (int w = 0; w < NE / 4; ++w) {
            uint32_t br[4], bi[4], bs[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int i = 4 * w + b;
                int Ry = dp4a_ss(dr[i].hi, wh, dp4a_us(dr[i].lo, wl, y0));  // A_r mod m (unreduced) on top of the bits of Y0
                if (WIDE) Ry = dp4a_ss(tr[i], wt, Ry);
                int ys = dp4a_ss(di[i].hi, wh, dp4a_us(di[i].lo, wl, Ry));  // A_r + A_i: the same weights for both parts
                if (WIDE) ys = dp4a_ss(ti[i], wt, ys);
                const int Iy = ys - Ry + y0;                                // A_i alone
                br[b] = sym_reduce_one(Ry, neg_m, inv_m, cq);
                bi[b] = sym_reduce_one(Iy, neg_m, inv_m, cq);
                bs[b] = sym_reduce_one(ys, neg_m, inv_m, cq);
            }
            rw[w] = pack4(br);
            iw[w] = pack4(bi);
            sw[w] = pack4(bs);
        }
        store_run<NE>(dst3 + (int64_t)j3 * plane_stride, rw);
        store_run<NE>(dst3 + (int64_t)(n3 + j3) * plane_stride, iw);
        store_run<NE>(dst3 + (int64_t)(2 * n3 + j3) * plane_stride, sw);
    }
}

// ---- floating-point inputs: persistent blocks, raw elements copied asynchronously into a two-stage ring (residues_common.cuh)
template <typename T, bool WIDE, int NMOD, bool HEX = false, bool NARROW = false>
__global__ void __launch_bounds__(kResThreads, kResBlocksPerSm) residues_fp_kernel(const T* __restrict__ X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K,
                                                                     int64_t Kp, int32_t* __restrict__ e, const ScaleFrom from,
                                                                     const __grid_constant__ ResidueTable tab, int8_t* __restrict__ planes,
                                                                     int64_t plane_rows) {
    using Raw = typename RawCplx<T>::type;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    wait_for_prior_kernels();
    Raw* ring = reinterpret_cast<Raw*>(smem_raw);
    constexpr int kStageElems = kResRows * kResRowStride;
    const int t = threadIdx.x;
    const int64_t ktiles = Kp / kResK;
    const int64_t total = ((R + kResRows - 1) / kResRows) * ktiles;
    const int64_t plane_stride = plane_rows * Kp;     // rows of a whole plane (R when the launch covers the operand, more for a row range)

    auto issue = [&](int64_t tile, int stage) {
        const int64_t row0 = (tile / ktiles) * kResRows, k0 = (tile % ktiles) * kResK;
        Raw* dst = ring + stage * kStageElems;
        if (!k_contiguous) {          // consecutive threads -> consecutive operand rows (rows of a column-major matrix)
            const int r = t & (kResRows - 1);
            const int64_t row = row0 + r;
#pragma unroll
            for (int kk = t / kResRows; kk < kResK; kk += kResThreads / kResRows) {
                const int64_t k = k0 + kk;
                const bool ok = row < R && k < K;
                cp_async_zfill<sizeof(Raw)>(dst + r * kResRowStride + kk + (kk >> 3), ok ? X + 2 * (row + k * ld) : X, ok);
            }
        } else {                      // consecutive threads -> consecutive k (columns of the matrix are contiguous)
            const int kk = t & (kResK - 1);
            const int64_t k = k0 + kk;
#pragma unroll
            for (int r = t / kResK; r < kResRows; r += kResThreads / kResK) {
                const int64_t row = row0 + r;
                const bool ok = row < R && k < K;
                cp_async_zfill<sizeof(Raw)>(dst + r * kResRowStride + kk + (kk >> 3), ok ? X + 2 * (k + row * ld) : X, ok);
            }
        }
        cp_async_commit();
    };

    int64_t tile = blockIdx.x;
    if (tile >= total) return;
    issue(tile, 0);
    for (int it = 0; tile < total; tile += gridDim.x, ++it) {
        const int64_t next = tile + gridDim.x;
        if (next < total) { issue(next, (it + 1) & 1); cp_async_wait_group<1>(); }
        else cp_async_wait_group<0>();
        __syncthreads();
        const Raw* src = ring + (it & 1) * kStageElems;
        const int64_t row0 = (tile / ktiles) * kResRows, k0 = (tile % ktiles) * kResK;
        const int g = t & (kResK / kResRun - 1), r = t / (kResK / kResRun);
        const int64_t row = row0 + r;
        if (row < R) {
            // the scale exponent: given, or formed here from the scan's maximum (and left in e for the post-processing)
            int ex;
            if (from.absmax) {
                ex = scale_exponent<T>(from.absmax[row], from.P, from.ck);
                if (k0 == 0 && g == 0) e[row] = ex;
            } else {
                ex = e[row];
            }
            // Narrow mode, ordinary exponents: x 2^-e is an exact FP64 product (or underflows towards zero, where the
            // truncation is zero anyway) and its truncation to int64 is one conversion; |x 2^-e| < 2^62 by the scaling rule.
            const bool fast = !WIDE && ex > -1000 && ex < 1000;
            const double scale = __longlong_as_double((long long)(1023 - (fast ? ex : 0)) << 52);
            Digits dr[kResRun], di[kResRun];
            uint32_t tr[WIDE ? kResRun : 1], ti[WIDE ? kResRun : 1];
#pragma unroll
            for (int i = 0; i < kResRun; ++i) {
                Raw v = src[r * kResRowStride + kResRun * g + g + i];
                if (conj) v.y = -v.y;                         // conjugated operand: the imaginary part changes sign before quantisation
                if (WIDE) {
                    uint32_t lr = 0, li = 0;
                    long long ur = 0, ui = 0;
                    if (ex != kExpNonFinite) {
                        if (HEX) {
                            __int128 su, sv;
                            quantise_hex((double)v.x, (double)v.y, ex, &su, &sv);
                            lr = (uint32_t)(unsigned __int128)su; ur = (long long)(su >> 32);
                            li = (uint32_t)(unsigned __int128)sv; ui = (long long)(sv >> 32);
                        } else {
                            quantise_part_wide<T>(v.x, ex, &lr, &ur);
                            quantise_part_wide<T>(v.y, ex, &li, &ui);
                        }
                    }
                    dr[i] = split_digits_wide(lr, ur, &tr[i]);
                    di[i] = split_digits_wide(li, ui, &ti[i]);
                } else {
                    long long qr = 0, qi = 0;
                    if (HEX) {
                        if (ex != kExpNonFinite) {
                            __int128 su, sv;
                            quantise_hex((double)v.x, (double)v.y, ex, &su, &sv);
                            qr = (long long)su;
                            qi = (long long)sv;
                        }
                    } else if (fast) {
                        qr = __double2ll_rz((double)v.x * scale);
                        qi = __double2ll_rz((double)v.y * scale);
                    } else if (ex != kExpNonFinite) {
                        qr = quantise_part<T>(v.x, ex);
                        qi = quantise_part<T>(v.y, ex);
                    }
                    if (NARROW) {              // |q| < 2^31: the low word plus 2^31 as four unsigned bytes
                        dr[i].lo = (uint32_t)(unsigned long long)qr ^ 0x80000000u; dr[i].hi = 0u;
                        di[i].lo = (uint32_t)(unsigned long long)qi ^ 0x80000000u; di[i].hi = 0u;
                    } else {
                        dr[i] = split_digits(qr);
                        di[i] = split_digits(qi);
                    }
                }
            }
            emit_run<kResRun, WIDE, NMOD, NARROW>(dr, di, tr, ti, tab, planes + row * Kp + k0 + kResRun * g, plane_stride);
        }
        __syncthreads();   // everyone is done with this stage before it is refilled
    }
}

constexpr size_t kResSmemBytes(size_t elem) { return (size_t)kResStages * kResRows * kResRowStride * elem; }


template <typename T>
cudaError_t launch_residues_fp(const T* X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K, int64_t Kp, int32_t* e,
                               const ResidueTable& tab, int width, int8_t* planes, cudaStream_t st, int* launches, int64_t plane_rows,
                               ScaleFrom from) {
    if (R <= 0 || Kp <= 0) return cudaSuccess;
    const bool wide = width == 1;
    const bool narrow = width == 2 && tab.n2 == tab.nmod;      // (the 3M moduli of the hybrid only come with wide values)
    constexpr size_t smem = kResSmemBytes(2 * sizeof(T));
    static bool attr_set_dev[kMaxDevices] = {};
    bool& attr_set = attr_set_dev[current_device_slot()];
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(residues_fp_kernel<T, false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess) err = cudaFuncSetAttribute(residues_fp_kernel<T, true, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
#define GEMM2M_RES_ATTR(N) if (err == cudaSuccess) err = cudaFuncSetAttribute(residues_fp_kernel<T, false, N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        GEMM2M_RES_ATTR(7) GEMM2M_RES_ATTR(8) GEMM2M_RES_ATTR(14) GEMM2M_RES_ATTR(15) GEMM2M_RES_ATTR(16)
#undef GEMM2M_RES_ATTR
        if (err == cudaSuccess) err = cudaFuncSetAttribute(residues_fp_kernel<T, false, 0, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess) err = cudaFuncSetAttribute(residues_fp_kernel<T, false, 7, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess) err = cudaFuncSetAttribute(residues_fp_kernel<T, false, 8, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    const int64_t total = ((R + kResRows - 1) / kResRows) * (Kp / kResK);
    const int64_t resident = (int64_t)cached_sm_count() * kResBlocksPerSm;
    const unsigned grid = (unsigned)(total < resident ? total : resident);
    // The modulus counts of the common use cases (7-8: single precision and the fastest settings, 14-16: double precision)
    // get a specialisation with the modulus loop unrolled: the per-modulus constants become constant-bank operands, which
    // saves two instructions per (element, modulus) -- 13 % of the kernel's time at 16 moduli.
    const int spec = (!wide && tab.n2 == tab.nmod) ? tab.nmod : 0;
    if (narrow) {
        // Values below 2^31 (few moduli: single precision, or the fastest double-precision settings): one dp4a per part
        if (spec == 7) launch_chained(residues_fp_kernel<T, false, 7, false, true>, grid, dim3(kResThreads), smem, st, X, ld, k_contiguous, conj, R, K, Kp, e, from, tab, planes, plane_rows ? plane_rows : R);
        else if (spec == 8) launch_chained(residues_fp_kernel<T, false, 8, false, true>, grid, dim3(kResThreads), smem, st, X, ld, k_contiguous, conj, R, K, Kp, e, from, tab, planes, plane_rows ? plane_rows : R);
        else launch_chained(residues_fp_kernel<T, false, 0, false, true>, grid, dim3(kResThreads), smem, st, X, ld, k_contiguous, conj, R, K, Kp, e, from, tab, planes, plane_rows ? plane_rows : R);
        ++*launches;
        return cudaGetLastError();
    }
    switch (spec) {
#define GEMM2M_RES_CASE(N) case N: launch_chained(residues_fp_kernel<T, false, N>, grid, dim3(kResThreads), smem, st, X, ld, k_contiguous, conj, R, K, Kp, e, from, tab, planes, plane_rows ? plane_rows : R); break;
        GEMM2M_RES_CASE(7) GEMM2M_RES_CASE(8) GEMM2M_RES_CASE(14) GEMM2M_RES_CASE(15) GEMM2M_RES_CASE(16)
#undef GEMM2M_RES_CASE
        default:
            if (wide) launch_chained(residues_fp_kernel<T, true, 0>, grid, dim3(kResThreads), smem, st, X, ld, k_contiguous, conj, R, K, Kp, e, from, tab, planes, plane_rows ? plane_rows : R);
            else launch_chained(residues_fp_kernel<T, false, 0>, grid, dim3(kResThreads), smem, st, X, ld, k_contiguous, conj, R, K, Kp, e, from, tab, planes, plane_rows ? plane_rows : R);
    }
    ++*launches;
    return cudaGetLastError();
}

// Eisenstein variant: the same kernel with the lattice rounding in front (complex double operands, 96-bit coordinates).
cudaError_t launch_residues_hex(const double* X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K, int64_t Kp, int32_t* e,
                                const ResidueTable& tab, bool wide, int8_t* planes, cudaStream_t st, int* launches, ScaleFrom from) {
    if (R <= 0 || Kp <= 0) return cudaSuccess;
    constexpr int64_t plane_rows = 0;
    constexpr size_t smem = kResSmemBytes(2 * sizeof(double));
    static bool attr_set_dev[kMaxDevices] = {};
    bool& attr_set = attr_set_dev[current_device_slot()];
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(residues_fp_kernel<double, true, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess) err = cudaFuncSetAttribute(residues_fp_kernel<double, false, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err == cudaSuccess) err = cudaFuncSetAttribute(residues_fp_kernel<double, false, 16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    const int64_t total = ((R + kResRows - 1) / kResRows) * (Kp / kResK);
    const int64_t resident = (int64_t)cached_sm_count() * kResBlocksPerSm;
    const unsigned grid = (unsigned)(total < resident ? total : resident);
    if (wide) launch_chained(residues_fp_kernel<double, true, 0, true>, grid, dim3(kResThreads), smem, st, X, ld, k_contiguous, conj, R, K, Kp, e, from, tab, planes, plane_rows ? plane_rows : R);
    else if (tab.nmod == 16) launch_chained(residues_fp_kernel<double, false, 16, true>, grid, dim3(kResThreads), smem, st, X, ld, k_contiguous, conj, R, K, Kp, e, from, tab, planes, plane_rows ? plane_rows : R);
    else launch_chained(residues_fp_kernel<double, false, 0, true>, grid, dim3(kResThreads), smem, st, X, ld, k_contiguous, conj, R, K, Kp, e, from, tab, planes, plane_rows ? plane_rows : R);
    ++*launches;
    return cudaGetLastError();
}

// ---- real floating-point inputs (real Ozaki-II scheme): one plane per modulus ---------------------------------------
template <int NE, bool WIDE>
__device__ __forceinline__ void emit_run_real(const Digits (&dr)[NE], const uint32_t* tr, const ResidueTable& tab, int8_t* dst, int64_t plane_stride) {
    const int nmod = tab.nmod;
#pragma unroll 1
    for (int j = 0; j < nmod; ++j) {
        const int neg_m = -tab.m[j], y0 = tab.magic[j];
        const float inv_m = tab.inv_m[j], cq = tab.cq[j];
        const uint32_t wl = tab.w_lo[j], wh = tab.w_hi[j], wt = WIDE ? tab.w_top[j] : 0u;
        uint32_t rw[NE / 4];
#pragma unroll
        for (int w = 0; w < NE / 4; ++w) {
            uint32_t br[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int i = 4 * w + b;
                int Ry = dp4a_ss(dr[i].hi, wh, dp4a_us(dr[i].lo, wl, y0));
                if (WIDE) Ry = dp4a_ss(tr[i], wt, Ry);
                br[b] = sym_reduce_one(Ry, neg_m, inv_m, cq);
            }
            rw[w] = pack4(br);
        }
        store_run<NE>(dst + (int64_t)j * plane_stride, rw);
    }
}

template <typename T, bool WIDE>
__global__ void __launch_bounds__(kResThreads, kResBlocksPerSm) residues_real_kernel(const T* __restrict__ X, int64_t ld, bool k_contiguous, int64_t R,
                                                                                   int64_t K, int64_t Kp, const int32_t* __restrict__ e,
                                                                                   const __grid_constant__ ResidueTable tab, int8_t* __restrict__ planes) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* ring = reinterpret_cast<T*>(smem_raw);
    constexpr int kStageElems = kResRows * kResRowStride;
    const int t = threadIdx.x;
    const int64_t ktiles = Kp / kResK;
    const int64_t total = ((R + kResRows - 1) / kResRows) * ktiles;
    const int64_t plane_stride = R * Kp;

    auto issue = [&](int64_t tile, int stage) {
        const int64_t row0 = (tile / ktiles) * kResRows, k0 = (tile % ktiles) * kResK;
        T* dst = ring + stage * kStageElems;
        if (!k_contiguous) {
            const int r = t & (kResRows - 1);
            const int64_t row = row0 + r;
#pragma unroll
            for (int kk = t / kResRows; kk < kResK; kk += kResThreads / kResRows) {
                const int64_t k = k0 + kk;
                const bool ok = row < R && k < K;
                cp_async_zfill<sizeof(T)>(dst + r * kResRowStride + kk + (kk >> 3), ok ? X + (row + k * ld) : X, ok);
            }
        } else {
            const int kk = t & (kResK - 1);
            const int64_t k = k0 + kk;
#pragma unroll
            for (int r = t / kResK; r < kResRows; r += kResThreads / kResK) {
                const int64_t row = row0 + r;
                const bool ok = row < R && k < K;
                cp_async_zfill<sizeof(T)>(dst + r * kResRowStride + kk + (kk >> 3), ok ? X + (k + row * ld) : X, ok);
            }
        }
        cp_async_commit();
    };

    int64_t tile = blockIdx.x;
    if (tile >= total) return;
    issue(tile, 0);
    for (int it = 0; tile < total; tile += gridDim.x, ++it) {
        const int64_t next = tile + gridDim.x;
        if (next < total) { issue(next, (it + 1) & 1); cp_async_wait_group<1>(); }
        else cp_async_wait_group<0>();
        __syncthreads();
        const T* src = ring + (it & 1) * kStageElems;
        const int64_t row0 = (tile / ktiles) * kResRows, k0 = (tile % ktiles) * kResK;
        const int g = t & (kResK / kResRun - 1), r = t / (kResK / kResRun);
        const int64_t row = row0 + r;
        if (row < R) {
            const int ex = __ldg(e + row);
            const bool fast = !WIDE && ex > -1000 && ex < 1000;
            const double scale = __longlong_as_double((long long)(1023 - (fast ? ex : 0)) << 52);
            Digits dr[kResRun];
            uint32_t tr[WIDE ? kResRun : 1];
#pragma unroll
            for (int i = 0; i < kResRun; ++i) {
                const T v = src[r * kResRowStride + kResRun * g + g + i];
                if (WIDE) {
                    uint32_t lr = 0;
                    long long ur = 0;
                    if (ex != kExpNonFinite) quantise_part_wide<T>(v, ex, &lr, &ur);
                    dr[i] = split_digits_wide(lr, ur, &tr[i]);
                } else {
                    long long qr = 0;
                    if (fast) qr = __double2ll_rz((double)v * scale);
                    else if (ex != kExpNonFinite) qr = quantise_part<T>(v, ex);
                    dr[i] = split_digits(qr);
                }
            }
            emit_run_real<kResRun, WIDE>(dr, tr, tab, planes + row * Kp + k0 + kResRun * g, plane_stride);
        }
        __syncthreads();
    }
}

template <typename T>
cudaError_t launch_residues_real(const T* X, int64_t ld, bool k_contiguous, int64_t R, int64_t K, int64_t Kp, const int32_t* e,
                                 const ResidueTable& tab, bool wide, int8_t* planes, cudaStream_t st, int* launches) {
    if (R <= 0 || Kp <= 0) return cudaSuccess;
    constexpr size_t smem = kResSmemBytes(sizeof(T));
    const int64_t total = ((R + kResRows - 1) / kResRows) * (Kp / kResK);
    const int64_t resident = (int64_t)cached_sm_count() * kResBlocksPerSm;
    const unsigned grid = (unsigned)(total < resident ? total : resident);
    if (wide) residues_real_kernel<T, true><<<grid, kResThreads, smem, st>>>(X, ld, k_contiguous, R, K, Kp, e, tab, planes);
    else residues_real_kernel<T, false><<<grid, kResThreads, smem, st>>>(X, ld, k_contiguous, R, K, Kp, e, tab, planes);
    ++*launches;
    return cudaGetLastError();
}
template cudaError_t launch_residues_real<double>(const double*, int64_t, bool, int64_t, int64_t, int64_t, const int32_t*, const ResidueTable&, bool, int8_t*, cudaStream_t, int*);

// ---- int8 Gaussian-integer inputs (no scaling): one 32 x 128 tile per block, loaded synchronously ---------------------
constexpr int kResIRows = 32, kResIRun = 16;
constexpr int kResIRowStride = kResK + kResK / kResIRun + 1;

__global__ void __launch_bounds__(kResIThreads) residues_int8_kernel(const int8_t* __restrict__ Xr, const int8_t* __restrict__ Xi, int64_t ld,
                                                                    bool k_contiguous, int64_t R, int64_t K, int64_t Kp,
                                                                    const __grid_constant__ ResidueTable tab, int8_t* __restrict__ planes) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    QPair* tile = reinterpret_cast<QPair*>(smem_raw);
    const int64_t row0 = (int64_t)blockIdx.y * kResIRows, k0 = (int64_t)blockIdx.x * kResK;
    const int t = threadIdx.x;
    auto fetch = [&](int r, int kk) -> QPair {
        const int64_t row = row0 + r, k = k0 + kk;
        QPair q{0, 0};
        if (row < R && k < K) {
            const int64_t idx = k_contiguous ? k + row * ld : row + k * ld;
            q.re = Xr[idx];
            q.im = Xi[idx];
        }
        return q;
    };
    if (!k_contiguous) {
        const int r = t & 31;
        for (int kk = t >> 5; kk < kResK; kk += kResIThreads / 32) tile[r * kResIRowStride + kk + (kk >> 4)] = fetch(r, kk);
    } else {
        const int kk = t & (kResK - 1);
        for (int r = t >> 7; r < kResIRows; r += kResIThreads / kResK) tile[r * kResIRowStride + kk + (kk >> 4)] = fetch(r, kk);
    }
    __syncthreads();
    const int g = t & 7, r = t >> 3;
    Digits dr[kResIRun], di[kResIRun];
#pragma unroll
    for (int i = 0; i < kResIRun; ++i) {
        const QPair q = tile[r * kResIRowStride + kResIRun * g + i + g];
        dr[i] = split_digits(q.re);
        di[i] = split_digits(q.im);
    }
    const int64_t row = row0 + r;
    if (row >= R) return;
    emit_run<kResIRun, false, 0, false>(dr, di, nullptr, nullptr, tab, planes + row * Kp + k0 + kResIRun * g, R * Kp);
}

cudaError_t launch_residues_int8(const int8_t* Xr, const int8_t* Xi, int64_t ld, bool k_contiguous, int64_t R, int64_t K, int64_t Kp,
                                 const ResidueTable& tab, int8_t* planes, cudaStream_t st, int* launches) {
    if (R <= 0 || Kp <= 0) return cudaSuccess;
    constexpr size_t smem = (size_t)kResIRows * kResIRowStride * sizeof(QPair);
    static bool attr_set_dev[kMaxDevices] = {};
    bool& attr_set = attr_set_dev[current_device_slot()];
    if (!attr_set) {
        cudaError_t err = cudaFuncSetAttribute(residues_int8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        attr_set = true;
    }
    dim3 grid((unsigned)(Kp / kResK), (unsigned)((R + kResIRows - 1) / kResIRows));
    residues_int8_kernel<<<grid, kResIThreads, smem, st>>>(Xr, Xi, ld, k_contiguous, R, K, Kp, tab, planes);
    ++*launches;
    return cudaGetLastError();
}

template cudaError_t launch_residues_fp<double>(const double*, int64_t, bool, bool, int64_t, int64_t, int64_t, int32_t*, const ResidueTable&, int, int8_t*, cudaStream_t, int*, int64_t, ScaleFrom);
template cudaError_t launch_residues_fp<float>(const float*, int64_t, bool, bool, int64_t, int64_t, int64_t, int32_t*, const ResidueTable&, int, int8_t*, cudaStream_t, int*, int64_t, ScaleFrom);

}  // namespace gemm2m

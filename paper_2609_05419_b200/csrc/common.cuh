// Shared declarations of the gemm2m CUDA library: constant tables passed to kernels by value,
// launch wrappers of each phase, and small device helpers.  Notation follows the paper:
// m_j = modulus (the first 22 are 2M moduli with s_j = their square root of -1; the hybrid of Section 3 appends up to four
// non-2M moduli that take 3M multiplication, Eq. (1)), M = product of the moduli in use.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gemm2m {

constexpr int kMax2M = 22;         // size of the greedy 2M modulus set in [1, 256] (Section 4)
constexpr int kMax3M = 4;          // non-2M moduli of the hybrid: 256, 253, 251, 249 (quantised values then still fit 96 bits)
constexpr int kMaxMod = kMax2M + kMax3M;
constexpr int kMaxEis = 23;        // moduli of the Eisenstein-integer variant (Sections 3.2, 4): M up to 2^160.9
constexpr int kMaxReal = 20;       // moduli of the real Ozaki-II scheme (Section 3.1; set of Section 4): M up to 2^155
constexpr int kMaxPlanes = 2 * kMax2M + 3 * kMax3M;   // residue planes per operand: two per 2M modulus, three per 3M modulus
constexpr int kMaxChunks = 5;      // 40-bit digits needed for M/2 < 2^184
constexpr int kChunkBits = 40;
constexpr int kExpNonFinite = INT32_MIN;   // scale-exponent sentinel: row/column holds an Inf or NaN

// Device status word values (written by kernels whose bounded waits give up).
constexpr int kDevOk = 0;
constexpr int kDevTimeoutProducer = 101, kDevTimeoutMma = 102, kDevTimeoutEpilogue = 103, kDevTimeoutSelfTest = 104;

// Number of 2M moduli among the first nmod, and of residue planes per operand.  Plane order: X+ of the 2M moduli, X- of the
// 2M moduli, then for the 3M moduli X_r, X_i, X_r + X_i (each group in modulus order).
__host__ __device__ inline int count_2m(int nmod) { return nmod < kMax2M ? nmod : kMax2M; }
__host__ __device__ inline int plane_count(int nmod) { return 2 * count_2m(nmod) + 3 * (nmod - count_2m(nmod)); }

// Per-modulus constants for the residue kernels, Eq. (2a).
// A quantised part x (two's complement, 64 bits; 96 bits in the wide mode used from 19-20 moduli on) is written as 4
// unsigned low bytes and 4 (8) balanced signed high digits; its residue is the dot product of those digits with
// w_b = sym(256^b mod m).
// The imaginary part uses s*w_b so that R + I = A_r + s A_i and R - I = A_r - s A_i (mod m).
struct ResidueTable {
    int32_t m[kMaxMod];
    float inv_m[kMaxMod];
    int32_t magic[kMaxMod];                    // bit pattern of the float 2^23 + u m, u m a multiple of 256: start of the real dp4a chain
    float cq[kMaxMod];                         // 1.5 2^23 - u: fma(y, inv_m, cq) = 1.5 2^23 + rint(x / m) for y = 2^23 + u m + x
    uint32_t w_lo[kMaxMod], w_hi[kMaxMod];     // int8 x4 each: sym(256^b mod m), b = 0..3 / 4..7
    uint32_t ws_lo[kMaxMod], ws_hi[kMaxMod];   // int8 x4 each: sym(s 256^b mod m)
    uint32_t w_top[kMaxMod], ws_top[kMaxMod];  // b = 8..11: only used when quantised values exceed 62 bits
    int32_t s[kMaxMod];
    int32_t xmax[kMaxMod];                     // bound on |real dp4a sum| + |imaginary dp4a sum| (host side only)
    int nmod, n2;                              // moduli in use; the first n2 are 2M moduli, the rest (ws = w) take 3M
};

// Modulus of every batch entry of a GEMM launch, for the epilogue (reduction of the int32 accumulators).
// The four bytes of the accumulator plus 2^31 are contracted with w (one dp4a starting at y0 = the bit pattern of the float
// Y0 minus sym(2^31 mod m)), then reduced as in the residue kernels: one FMA with cq, one integer multiply-add.
struct ModTable {
    int32_t m[kMaxPlanes];
    float inv_m[kMaxPlanes];
    uint32_t w[kMaxPlanes];        // int8 x4: sym(256^b mod m), b = 0..3
    int32_t y0[kMaxPlanes];
    float cq[kMaxPlanes];
    int nplanes;
};

// CRT constants for the floating-point post-processing (Eq. (2c) folded into the CRT weights):
//   X_r = sum_j (c-_j + c+_j) Gr_j  (mod M),  Gr_j = sym(2^-1 q_j mod m_j) (M/m_j)
//   X_i = sum_j (c-_j - c+_j) Gi_j  (mod M),  Gi_j = sym(s_j 2^-1 q_j mod m_j) (M/m_j)
// with q_j = (M/m_j)^-1 mod m_j.  For a 3M modulus (j >= n2) the planes hold P1, P2, P3 of Eq. (1) and
//   X_r += (P1 - P2) G_j,  X_i += (P3 - P1 - P2) G_j,  G_j = sym(q_j mod m_j) (M/m_j)   (stored in both gr and gi).
// Each weight is stored as signed base-2^40 digits held in doubles, so
// that every digit-column sum is an exact integer below 2^53.  The multiple of M to remove is estimated from the
// two leading digit-column sums: t = rint(S_top q_hi + S_(top-1) q_lo), q_hi = 2^(40 top)/M, q_lo = q_hi 2^-40.
struct CrtTable {
    double gr[kMaxMod][kMaxChunks];
    double gi[kMaxMod][kMaxChunks];
    double Mc[kMaxChunks];                     // digits of M
    double q_hi, q_lo;
    double im_hi, im_lo;                       // Eisenstein variant: the imaginary part is V (im_hi + im_lo); 0 = no factor
    int nmod, n2, nchunks;
    int re_shift;                              // Eisenstein variant: the real part is U 2^re_shift
};

// Operands of the post-processing of the complex GEMMs, where the digit-column sums of the CRT are an 8-bit contraction on
// the tensor cores: per output element, [residues of all planes, + 128] x [base-256 digits of the folded CRT weights mod M].
//   X_r = sum_planes c_p Wr_p,  X_i = sum_planes c_p Wi_p  (mod M)
// with, for a 2M modulus j (planes C+_j and C-_j; Eq. (2c) folded in), Wr = Gr_j for both and Wi = -Gi_j / +Gi_j; for a 3M
// modulus (planes P1, P2, P3 of Eq. (1)) Wr = +G, -G, 0 and Wi = -G, -G, +G.  Every weight is reduced to [0, M) and written in
// bytes, W = sum_p d_p 256^p, p < 4 nb (nb even); with the residues moved to [0, 255] as well every digit-column sum is a
// non-negative integer.  The contraction runs as warp-level m16n8k32 MMAs: ks K-steps of 32 planes, nb blocks of 8 columns;
// bfrag holds the B-operand registers of every lane, [(s nb + q) 2 + h][lane], so that the digit column sums of one part land
// in the accumulators of two neighbouring lanes (see post_fp.cu for the column order).
constexpr int kPostMaxNB = 6, kPostMaxKS = 2;
constexpr int kPostFragWords = kPostMaxKS * kPostMaxNB * 2 * 32;
struct PostConsts {
    double Mc[kPostMaxNB];                     // M = sum_k Mc[k] 2^(32k), lower digits balanced in [-2^31, 2^31), each stored times 2^(32k)
    double off[2][kPostMaxNB];                 // per part: (1.5 2^52 + digit k of 128 sum_planes W_p) 2^(32k), what comes off chunk k
    double inv_M;                              // 1 / M
    double im_hi, im_lo;                       // Eisenstein variant: the imaginary part is V (im_hi + im_lo); 0 = no factor
    int re_shift;                              // Eisenstein variant: the real part is U 2^re_shift
    int planes, ks, nb;
};
struct PostMmaTable {
    PostConsts c;
    int nmod;                                  // moduli the table was built for
    uint32_t bfrag[kPostFragWords];            // host copy; launch_post_operands writes it to device memory
    uint8_t digit[2][32 * kPostMaxKS][4 * kPostMaxNB];   // [part][plane (K slot)][p]: the digits themselves (host side; for tests)
};

// CRT constants for the exact int64 result (nmod <= 8, M < 2^62).
struct CrtTableInt {
    int64_t W[8];          // M / m_j
    int32_t gr[8], gi[8];  // sym(2^-1 q_j), sym(s_j 2^-1 q_j)  (mod m_j)
    int32_t m[8];
    int64_t M;
    int nmod;
};

struct ScaleTargets { int Pt, PA, PB, ck; };

// Where a residue kernel takes its scale exponents from: the array e (absmax == null), or the scan's per-row maxima, from
// which it forms e = floor(log2 mu) + 1 + c_k - P itself and leaves it in e (one kernel launch less per operand).
struct ScaleFrom {
    const unsigned long long* absmax = nullptr;
    int P = 0, ck = 0;
};

// Function attributes (dynamic shared memory size, cluster occupancy) belong to a device: launchers cache "done" per device.
constexpr int kMaxDevices = 64;
// Programmatic dependent launch: a kernel launched through launch_chained may be made resident while the kernel before it on
// the stream is still draining; it calls wait_for_prior_kernels() before its first access to global memory, which returns
// once every earlier kernel of the stream has completed and its writes are visible.  Every kernel launched this way makes
// that call, so the order of the stream's memory effects is the usual one; what overlaps is launch latency and block
// set-up.  gemm2m_debug_set_chained_launch(0) falls back to plain launches.  (A kernel that follows a memset or an event is
// launched plainly.)
bool chained_launch_enabled();
#ifdef __CUDACC__
__device__ __forceinline__ void wait_for_prior_kernels() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// (Releasing the next kernel early, with griddepcontrol.launch_dependents at the top of each kernel, measured slower than the
// implicit release at block exit: 42 against 39 us per call at 512^3, 97 against 95 us at 1024^3.)
template <typename... P, typename... A>
inline cudaError_t launch_chained(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A&&... args) {
    cudaLaunchConfig_t c = {};
    c.gridDim = grid;
    c.blockDim = block;
    c.dynamicSmemBytes = smem;
    c.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    c.attrs = at;
    c.numAttrs = chained_launch_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&c, kernel, P(args)...);
}
#endif

inline int current_device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
    return dev;
}

// ---- host-side table builders (tables.cu) ----
int modulus_value(int j);
int modulus_root(int j);
void build_residue_table(int nmod, ResidueTable* t);
double residue_reduction_margin(const ResidueTable& t, int j);
// per_plane: one entry per residue plane in plane order (complex GEMM); otherwise one entry per modulus (rank-k family).
void build_mod_table(int nmod, bool per_plane, ModTable* t);
void build_crt_table(int nmod, CrtTable* t);
void build_crt_table_int(int nmod, CrtTableInt* t);
void build_post_mma_table(int nmod, PostMmaTable* t);
void build_post_mma_table_eis(int nmod, PostMmaTable* t);
// Rank-k family (Section 5): the planes are the C+ planes read directly (K slots 0 .. nmod-1) and read mirrored, as C- = C+^T
// (K slots H .. H + nmod - 1 with H = nmod rounded up to 16, so that every 16-slot half of K holds planes of one kind).
void build_post_mma_table_herk(int nmod, PostMmaTable* t);
ScaleTargets scale_targets(int nmod, int64_t k, bool herk);
// The same for the real Ozaki-II scheme (dgemm_ozaki2): moduli 256, 255, 253, ..., one residue plane per modulus.
int real_modulus_value(int j);
void build_residue_table_real(int nmod, ResidueTable* t);
void build_mod_table_real(int nmod, ModTable* t);
void build_crt_table_real(int nmod, CrtTable* t);
ScaleTargets scale_targets_real(int nmod, int64_t k);
// The same for the Eisenstein-integer variant (zgemm2m_eisenstein): moduli 247, 241, 229, ..., two planes per modulus, the
// residue table's s_j = 2 (cube root) + 1, a square root of -3.
int eis_modulus_value(int j);
int eis_cube_root(int j);
void build_residue_table_eis(int nmod, ResidueTable* t);
void build_mod_table_eis(int nmod, ModTable* t);
void build_crt_table_eis(int nmod, CrtTable* t);
ScaleTargets scale_targets_eis(int nmod, int64_t k);
int64_t gemm_k_limit_eis();
int64_t gemm_k_limit_real();
int64_t gemm_k_limit(int nmod);     // largest K for which K max|residue|^2 fits int32

// ---- phase launchers (scan.cu, residues.cu, post.cu) ----
// Exponent scan: largest |Re|,|Im| bit pattern per row of a column-major matrix (rows x cols, ld).
template <typename T> cudaError_t launch_scan_rows(const T* X, int64_t rows, int64_t cols, int64_t ld, uint64_t* absmax, cudaStream_t st, int* launches, bool chained = false);
// The same per column.  (chained: the launch directly follows another kernel on the stream, see launch_chained.)
template <typename T> cudaError_t launch_scan_cols(const T* X, int64_t rows, int64_t cols, int64_t ld, uint64_t* absmax, cudaStream_t st, int* launches, bool chained = false);
template <typename T> cudaError_t launch_exponents(const uint64_t* absmax, int64_t count, int P, int ck, int32_t* e, cudaStream_t st, int* launches);
// 2-norm scaling rule: second pass over X (rows x cols, ld) summing the squared fixed-point magnitudes per row (per_row) or
// per column into qsum (zeroed by the caller), then e = x + 1 - P + ceil(log4 Q) - 20 with x from absmax.
template <typename T> cudaError_t launch_exponents_2norm(const T* X, int64_t rows, int64_t cols, int64_t ld, bool per_row, const uint64_t* absmax,
                                                         uint64_t* qsum, int P, int32_t* e, cudaStream_t st, int* launches);
// Quantise + residues.  k_contiguous = false: operand row r is row r of the column-major matrix X (A: m x k);
// true: operand row r is column r of X (B: k x n).
// conj: the operand is the complex conjugate of X.  wide = quantised values may need more than 62 bits (P - c_k > 62).
cudaError_t launch_residues_hex(const double* X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K, int64_t Kp, int32_t* e,
                                const ResidueTable& tab, bool wide, int8_t* planes, cudaStream_t st, int* launches, ScaleFrom from = ScaleFrom());
// width: 0 = quantised values of up to 62 bits, 1 = wide (up to 94 bits), 2 = narrow (|value| < 2^31: half the byte-weight chain).
// plane_rows: rows of a whole plane when the launch covers a row range of the operand only (X, e and planes then point at the
// first row of the range); 0 = R.
template <typename T> cudaError_t launch_residues_fp(const T* X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K, int64_t Kp,
                                                     int32_t* e, const ResidueTable& tab, int width, int8_t* planes, cudaStream_t st, int* launches,
                                                     int64_t plane_rows = 0, ScaleFrom from = ScaleFrom());
cudaError_t launch_residues_int8(const int8_t* Xr, const int8_t* Xi, int64_t ld, bool k_contiguous, int64_t R, int64_t K, int64_t Kp,
                                 const ResidueTable& tab, int8_t* planes, cudaStream_t st, int* launches);
// Columns [j_begin, j_end) of C only (n stays the full column count: it fixes the plane stride).
// alpha, beta: host pointers to (re, im) pairs, or null for alpha = 1 / beta = 0: C = alpha X + beta C.
// dev_frags: device copy of tab.bfrag, written earlier on an ordered stream by launch_post_operands (kPostFragWords words).
cudaError_t launch_post_operands(const PostMmaTable& tab, uint32_t* dev_frags, cudaStream_t st, int* launches);
template <typename T> cudaError_t launch_post_fp(const int8_t* cpm, int64_t ldp, int64_t m, int64_t n, int64_t j_begin, int64_t j_end, const int32_t* eA, const int32_t* eB,
                                                 const PostMmaTable& tab, const uint32_t* dev_frags, T* C, int64_t ldc, const double* alpha, const double* beta,
                                                 cudaStream_t st, int* launches);
// Real Ozaki-II scheme (Section 3.1): scans, residues (one plane per modulus) and post-processing of real matrices.
template <typename T> cudaError_t launch_scan_real(const T* X, int64_t rows, int64_t cols, int64_t ld, bool per_row, uint64_t* absmax, cudaStream_t st, int* launches);
template <typename T> cudaError_t launch_residues_real(const T* X, int64_t ld, bool k_contiguous, int64_t R, int64_t K, int64_t Kp, const int32_t* e,
                                                       const ResidueTable& tab, bool wide, int8_t* planes, cudaStream_t st, int* launches);
cudaError_t launch_post_real(const int8_t* cp, int64_t ldp, int64_t m, int64_t n, int64_t j_begin, int64_t j_end, const int32_t* eA, const int32_t* eB,
                             const CrtTable& tab, double* C, int64_t ldc, cudaStream_t st, int* launches);
// C = beta C (the alpha = 0 case of the extended interface); beta = host pointer to (re, im) or null for 0.
template <typename T> cudaError_t launch_scale_c(T* C, int64_t m, int64_t n, int64_t ldc, const double* beta, cudaStream_t st, int* launches);
// real_out: C is a real matrix (SYRK / SYR2K through Z = A1 + i A2): only the real part is formed and stored.
// Rows [i_begin, i_end) of the lower triangle only (i_begin a multiple of 64): they need the GEMM output rows below i_end.
cudaError_t launch_post_herk(const int8_t* cp, int64_t ldp, int64_t n, int64_t i_begin, int64_t i_end, const int32_t* eA, const PostMmaTable& tab,
                             const uint32_t* dev_frags, double* C, int64_t ldc, bool real_out, cudaStream_t st, int* launches);
// Z[i, p] = X[i, p] + i X[i, p + k2] for p < k2 = ceil(k / 2) (zero beyond column k): the complex matrix whose HERK is the SYRK of X.
cudaError_t launch_pack_real_pair(const double* X, int64_t ld, int64_t n, int64_t k, double* Z, cudaStream_t st, int* launches);
cudaError_t launch_post_int(const int8_t* cpm, int64_t ldp, int64_t m, int64_t n, const CrtTableInt& tab, int64_t* Cr, int64_t* Ci,
                            int64_t ldc, cudaStream_t st, int* launches);

// ---- int8 GEMM (gemm_i8_2cta.cu; check kernel: gemm_check.cu) ----
// For each batch b in [0, nbatch): out[b][r][c] = sym( sum_k rowop[b + row_plane0][r][k] * colop[b + col_plane0][c][k]  mod (modulus of batch entry b) ),
// r < R, c < Cn, k < Kp (zero padded); planes are [*][rows][Kp] int8; out planes are [R][ldp] int8.
struct GemmArgs {
    const int8_t* rowop; const int8_t* colop;
    int64_t R, Cn, Kp;
    int64_t row_begin, row_end;       // rows of the row operand handled by this launch (multiples of 256, or R)
    int row_planes, col_planes;       // number of planes behind each pointer (for the tensor maps)
    int row_plane0, col_plane0, nbatch;
    int8_t* out; int64_t ldp;
    int accumulate;                   // add to the residues already stored in `out` (second product of a rank-2k update)
    ModTable mods;
    int* dev_status;
};
cudaError_t launch_gemm_tcgen05_pair(const GemmArgs& a, int64_t k_limit, int sm_count, cudaStream_t st, int* launches);   // CTA pairs
cudaError_t launch_gemm_check(const GemmArgs& a, int64_t k_limit, cudaStream_t st, int* launches);
// One thread waits, with the GEMM kernel's bounded wait and a budget of budget_ns, on a barrier nobody arrives on: the wait
// gives up, records its code in *dev_status and the kernel returns.
cudaError_t launch_wait_selftest(int* dev_status, unsigned long long budget_ns, cudaStream_t st);

}  // namespace gemm2m

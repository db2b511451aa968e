/*
 * gemm2m -- complex matrix multiplication by 2M multiplication + the Ozaki-II scheme, for NVIDIA B200 (sm_100a).
 *
 * Complex GEMM with only two real int8 GEMMs per modulus:
 *   1. per-row (A) / per-column (B) power-of-two scale factors, entries truncated to Gaussian integers
 *      (Algorithm 1 steps 2-3; Section 3.1 for the real scheme);
 *   2. for each 2M modulus m_j (odd, s_j^2 = -1 mod m_j; Section 2, set of Section 4) the residues
 *      A+- = A_r +- s_j A_i, B+- = B_r +- s_j B_i (mod m_j), Eq. (2a), kept as symmetric int8;
 *   3. the two real products C+- = A+- B+- (mod m_j), Eq. (2b), on the int8 tensor cores;
 *   4. C = 2^-1 (C- + C+) + i s_j 2^-1 (C- - C+) (mod m_j), Eq. (2c); CRT over j (Section 3.1; Algorithm 1
 *      step 5); lift to the symmetric range (step 6); multiply by sigma_i tau_j (step 7).
 *
 * Beyond that path the library offers, each documented at its declaration: the same call on host operands with the
 * transfers overlapped inside it (zgemm2m_host), the hybrid 2M/3M moduli (nmod 23..26), the
 * BLAS-style forms with op(A), op(B), alpha, beta (zgemm2m_ex, cgemm2m_ex), the rank-k family of Section 5 (zherk2m,
 * zher2k2m, dsyrk2m, dsyr2k2m), an optional tighter choice of the scale factors (gemm2m_set_scaling), the real
 * Ozaki-II scheme of Section 3.1 (dgemm_ozaki2) and the Eisenstein-integer variant of Sections 3.2 and 4
 * (zgemm2m_eisenstein).
 *
 * Conventions for every entry point
 *   - BLAS-3 style as in the paper's problem statement (Section 1: A in C^{m x k}, B in C^{k x n}; Section 6:
 *     alpha = 1, beta = 0): column-major, complex numbers interleaved (re, im), leading dimensions counted in
 *     elements (complex elements for complex matrices), no transposition arguments, C is overwritten.
 *   - All matrix pointers are DEVICE pointers owned by the caller (zgemm2m_host alone takes host pointers).  The library never allocates or frees device
 *     memory inside a call; it uses the caller-provided workspace registered with gemm2m_set_workspace().
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream) and
 *     return immediately.  The return value is a gemm2m_status; it is the only error channel.  Every kernel of a call
 *     runs on `stream`, in order (some are launched as programmatic dependents of the kernel before them: such a kernel may
 *     become resident early, and waits on the device for every earlier kernel before it touches global memory).  (zgemm2m_host alone uses library-owned streams, for its copies and the work that runs
 *     beside them, forked from and joined back into `stream` with events: work enqueued on `stream` after the call still
 *     sees the finished result.  So does every entry point while gemm2m_debug_set_overlap(1) is in force.)
 *   - Because a call only enqueues (kernels, memsets, event records and waits), it can be captured into a CUDA graph
 *     and replayed; a library-owned stream joins the capture through its fork/join events.  Make one call outside any
 *     capture first: it creates such streams and events, and leaves in the workspace the constant operand of the
 *     post-processing, which later calls with the same modulus count reuse.  (gemm2m_set_profiling must be off during a capture.)
 *   - The workspace belongs to the library while it is registered: besides the status word it keeps that operand between
 *     calls.  Register it again (gemm2m_set_workspace) after writing to it.
 *   - Argument errors are detected on the host before anything is launched.  m, n or k equal to 0 is valid:
 *     nothing is computed for m = 0 or n = 0, and C is set to zero for k = 0.
 *   - `nmod` selects the first nmod moduli of the set of Section 4 (241, 233, 229, 221, 205, ... , 37, 29; 22 in
 *     all).  More moduli = larger M = more accuracy and proportionally more work.  16 gives about double
 *     precision accuracy for zgemm2m/zherk2m, 7 about single precision for cgemm2m.
 *   - Hybrid 2M/3M (remark after Algorithm 1; Section 4, last paragraph but one): zgemm2m and cgemm2m also accept
 *     nmod = 23 ... 26.  The moduli beyond the 22nd are the non-2M moduli 256, 253, 251, 249 (the next numbers of the
 *     greedy walk down from 256 that are coprime to everything chosen before); each of them takes 3M multiplication,
 *     Eq. (1), applied after the reduction modulo m: three real int8 GEMMs A_r B_r, A_i B_i, (A_r + A_i)(B_r + B_i).
 *     M reaches about 2^184; useful when a row of A or a column of B spans many binary orders of magnitude.  The
 *     rank-k family and gemm2m_gaussian_int take 2M moduli only.
 *   - One call at a time per workspace: calls that share a workspace must be ordered on the GPU (same stream).
 *   - Entry points may be called from several host threads, on the same or on different GPUs; they serialise on one
 *     library-wide mutex for the time it takes to enqueue a call (the GPU work of calls on different GPUs still overlaps).
 *   - Non-finite inputs: a row of A (column of B) that contains an Inf or NaN yields NaN in the whole
 *     corresponding row (column) of C; no error is reported.
 */
#ifndef GEMM2M_H
#define GEMM2M_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GEMM2M_OK = 0,
    GEMM2M_ERR_ARG = 1,            /* negative size, leading dimension too small, null pointer with non-empty matrix */
    GEMM2M_ERR_NMOD = 2,           /* nmod outside [1, 26] (zgemm2m, cgemm2m) or [1, 22] (rank-k family), or > 8 for gemm2m_gaussian_int */
    GEMM2M_ERR_WORKSPACE = 3,      /* no workspace registered or too small; nothing was launched */
    GEMM2M_ERR_CUDA = 4,           /* a CUDA runtime/driver call failed (see gemm2m_last_cuda_error) */
    GEMM2M_ERR_ARCH = 5,           /* current device is not compute capability 10.0 */
    GEMM2M_ERR_DEVICE_TIMEOUT = 6  /* a bounded device-side wait gave up (reported by gemm2m_device_status) */
} gemm2m_status;

typedef enum {
    GEMM2M_OP_GAUSSIAN_INT = 0, GEMM2M_OP_ZGEMM = 1, GEMM2M_OP_CGEMM = 2, GEMM2M_OP_ZHERK = 3,
    GEMM2M_OP_ZHER2K = 4, GEMM2M_OP_DSYRK = 5, GEMM2M_OP_DSYR2K = 6, GEMM2M_OP_DGEMM_OZAKI2 = 7,
    GEMM2M_OP_ZGEMM_EISENSTEIN = 8, GEMM2M_OP_ZGEMM_HOST = 9
} gemm2m_op;

/* Human-readable name of a status code (static string). */
const char* gemm2m_status_string(int status);
/* Text of the last CUDA error seen by this thread's calls (static/thread-local string, never NULL). */
const char* gemm2m_last_cuda_error(void);

/* Number of moduli available to zgemm2m / cgemm2m (26): the 2M moduli followed by the 3M moduli of the hybrid. */
int gemm2m_max_moduli(void);
/* Number of 2M moduli available (22): the greedy coprime set in [1, 256] of Section 4. */
int gemm2m_max_2m_moduli(void);
/* j-th modulus (0-based; the 2M moduli in descending order, then the 3M moduli) and its smallest positive square root
 * of -1 (Section 2), 0 for a 3M modulus.  Host pointers. */
int gemm2m_modulus(int j, int* m, int* s);

/* Bytes of device workspace a call of `op` with these sizes needs (for the rank-k family pass m = n).  0 on bad arguments. */
size_t gemm2m_workspace_bytes(int op, int64_t m, int64_t n, int64_t k, int nmod);
/* Register a caller-owned device buffer (256-byte aligned) of the CURRENT device; later calls made while that device is
 * current use it (one workspace per device; the library's side stream and events are per device too).  Passing (NULL, 0)
 * unregisters.  The buffer must stay valid until the last call using it has finished. */
int gemm2m_set_workspace(void* dev_ptr, size_t bytes);

/* Gaussian-integer product by 2M multiplication (Section 2, Eq. (2a)-(2c)) and CRT over nmod <= 8 moduli.
 * Ar, Ai: m x k int8 (lda >= m); Br, Bi: k x n int8 (ldb >= k); Cr, Ci: m x n int64 (ldc >= m), overwritten with
 * the representative of the exact product modulo M = m_1 ... m_nmod in [-(M-1)/2, (M-1)/2] -- the exact product
 * itself whenever 2 max|c| < M (first paragraph of Section 2). */
int gemm2m_gaussian_int(int64_t m, int64_t n, int64_t k,
                        const int8_t* Ar, const int8_t* Ai, int64_t lda,
                        const int8_t* Br, const int8_t* Bi, int64_t ldb,
                        int64_t* Cr, int64_t* Ci, int64_t ldc, int nmod, void* stream);

/* C = A B in complex double precision by Algorithm 1 ("2M Ozaki-II").  A: m x k, B: k x n, C: m x n, interleaved
 * complex128, lda >= m, ldb >= k, ldc >= m. */
int zgemm2m(int64_t m, int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb,
            double* C, int64_t ldc, int nmod, void* stream);

/* zgemm2m on HOST operands (the end-to-end form): A_host, B_host, C_host are host pointers with the layout of zgemm2m's A,
 * B, C; the transfers are part of the call and overlap its kernels.  A is uploaded first (every GEMM needs all of its
 * residue planes); B is uploaded in up to 32 column panels, and each panel is scanned, reduced to residues, multiplied and
 * post-processed while the next one is on the bus (the scale factor of a column of B depends on that column alone, so the
 * result is bit for bit zgemm2m's); each finished column panel of C is downloaded beside the next panel's work.  Copies run
 * on two library-owned streams, one per direction, ordered against `stream` by events; the call is complete on `stream`
 * when the last panel of C has arrived, and C_host, A_host, B_host must stay valid and unmodified until then.
 * Page-locked host memory (cudaHostAlloc / cudaHostRegister, torch pin_memory) is needed for the copies to be asynchronous
 * and to overlap; pageable memory works but serialises.  The workspace additionally holds compact device copies of A, B and
 * C: gemm2m_workspace_bytes(GEMM2M_OP_ZGEMM_HOST, ...).  Always the max-based scaling rule; nmod up to 26. */
int zgemm2m_host(int64_t m, int64_t n, int64_t k, const double* A_host, int64_t lda, const double* B_host, int64_t ldb,
                 double* C_host, int64_t ldc, int nmod, void* stream);

/* The same for complex single precision (interleaved complex64). */
int cgemm2m(int64_t m, int64_t n, int64_t k, const float* A, int64_t lda, const float* B, int64_t ldb,
            float* C, int64_t ldc, int nmod, void* stream);

/* BLAS-style extended forms (the paper fixes alpha = 1, beta = 0 and untransposed operands, Section 6; these follow
 * the ZGEMM / CGEMM conventions beyond that): C = alpha op(A) op(B) + beta C with op(X) = X ('N'), X^T ('T') or X^H ('C'),
 * op(A) m x k, op(B) k x n.  A is stored m x k ('N', lda >= m) or k x m (lda >= k); B is stored k x n ('N', ldb >= k) or
 * n x k (ldb >= n).  alpha, beta: HOST pointers to one complex number (re, im); NULL means alpha = 1 / beta = 0.
 * The product op(A) op(B) is formed exactly as by zgemm2m (a transposed operand is only read in the other orientation; a
 * conjugated one changes the sign of its imaginary parts before quantisation), rounded once, and then combined with
 * alpha, beta and the old C in working precision with fused multiply-adds.  beta = 0: C is not read; alpha = 0: A and B
 * are not read and C = beta C.  A bad trans character returns GEMM2M_ERR_ARG. */
int zgemm2m_ex(char transa, char transb, int64_t m, int64_t n, int64_t k, const double* alpha, const double* A, int64_t lda,
               const double* B, int64_t ldb, const double* beta, double* C, int64_t ldc, int nmod, void* stream);
int cgemm2m_ex(char transa, char transb, int64_t m, int64_t n, int64_t k, const float* alpha, const float* A, int64_t lda,
               const float* B, int64_t ldb, const float* beta, float* C, int64_t ldc, int nmod, void* stream);

/* Choice of the scale factors sigma_i, tau_j of zgemm2m / cgemm2m and their _ex forms (Algorithm 1 step 2; the paper
 * leaves it to the literature).  Both choices are powers of two that make the 2-norm of every scaled row of A at most
 * 2^P_A and of every scaled column of B at most 2^P_B, P_A + P_B = floor(log2((M-1)/2)), which by Cauchy-Schwarz keeps every
 * entry of the integer product inside the range the CRT can represent.
 *   0 (default): from the largest |Re| or |Im| of the row, times sqrt(2k): one pass over the operands;
 *   1: from an upper bound of the row's 2-norm itself (sum of the squares of the parts, each rounded up to 20 fractional
 *      bits below the largest one's binade, in 64-bit integers): a second pass over A and B, and in return 3 to 6 more
 *      bits of each operand survive the truncation, about what one more modulus buys.  Falls back to 0 for k > 2^22.
 * Process-wide; takes effect with the next call.  The rank-k family always uses 0. */
int gemm2m_set_scaling(int mode);

/* The real Ozaki-II scheme the paper builds on and compares with (Section 3.1; Section 6 finds one ZGEMM to cost about
 * 2.16 real Ozaki-II DGEMMs): C = A B for REAL double matrices (A: m x k, lda >= m; B: k x n, ldb >= k; C: m x n, ldc >= m, real doubles),
 * with ONE real int8 GEMM per modulus of the real modulus set of Section 4 (256, 255, 253, 251, 247, 241, ...; every
 * coprime number qualifies, nmod <= 20, 15 give M ~ 2^117).  Same readings as zgemm2m: power-of-two scale factors from
 * the largest magnitude of a row / column times sqrt(k), truncation, symmetric residues, one rounding.  Workspace:
 * gemm2m_workspace_bytes(GEMM2M_OP_DGEMM_OZAKI2, ...). */
int dgemm_ozaki2(int64_t m, int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc,
                 int nmod, void* stream);

/* The Eisenstein-integer analogue of zgemm2m that Sections 3.2 and 4 point out: the Gaussian integers are replaced by
 * Z[w], w = exp(2 pi i/3), whose 2M moduli are the products of primes congruent to 1 mod 3 (greedy coprime set below 256:
 * 247, 241, 229, 223, 217, 211, 199, ..., 43, 37; nmod <= 23, M up to 2^160.9 against 2^152 for the Gaussian set).
 * Same interface, layout, workspace rules and GEMMs as zgemm2m / zgemm2m_ex (two real int8 GEMMs per modulus); different:
 *   - quantisation rounds each scaled entry to the NEAREST point of the hexagonal lattice, held as (u + v sqrt(-3))/2 with
 *     u = v (mod 2).  The decision is taken in fixed point (32 fraction bits, 2/sqrt(3) as a 128-bit constant), so that it is
 *     reproducible bit for bit; it differs from the exact nearest point only within 2^-30 of a cell boundary;
 *   - the residues are u +- d_j v with d_j = 2 s_j + 1 a square root of -3 modulo m_j (s_j^2 + s_j + 1 = 0), twice the images
 *     of the entry under w -> s_j and w -> s_j^2; the factor 4 this leaves in the products is folded into the CRT weights;
 *   - the scale factors use c_k = ceil(log2(5k)/2) (lattice rounding can move a point outwards; the coordinates of a
 *     product are bounded by twice its modulus), and P_B - c_k >= 2 is required: too few moduli for k give GEMM2M_ERR_NMOD;
 *   - the lifted result (U + V sqrt(-3))/2 is converted with one rounding per part: Re = U/2, Im = V sqrt(3)/2 (the
 *     irrational factor as a double-double).
 * The always-on max-based scaling rule is used (gemm2m_set_scaling does not apply).  Workspace:
 * gemm2m_workspace_bytes(GEMM2M_OP_ZGEMM_EISENSTEIN, ...). */
int zgemm2m_eisenstein(int64_t m, int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C,
                       int64_t ldc, int nmod, void* stream);
int zgemm2m_eisenstein_ex(char transa, char transb, int64_t m, int64_t n, int64_t k, const double* alpha, const double* A,
                          int64_t lda, const double* B, int64_t ldb, const double* beta, double* C, int64_t ldc, int nmod,
                          void* stream);
/* Size of the Eisenstein modulus set (23) and its j-th modulus with the smallest s_j > 1, s_j^2 + s_j + 1 = 0 (mod m_j). */
int gemm2m_max_eisenstein_moduli(void);
int gemm2m_eisenstein_modulus(int j, int* m, int* s);

/* Hermitian rank-k update C = A A^H (Section 5, HERK) with ONE real int8 GEMM per modulus: C+ = A+ A-^T and
 * C- = C+^T.  A: n x k complex128 (lda >= n).  Only the lower triangle of C (n x n, ldc >= n) including the
 * diagonal is written; diagonal imaginary parts are exactly 0; the strict upper triangle is not touched. */
int zherk2m(int64_t n, int64_t k, const double* A, int64_t lda, double* C, int64_t ldc, int nmod, void* stream);

/* Hermitian rank-2k update C = A B^H + B A^H (Section 5, HER2K) with TWO real int8 GEMMs per modulus instead of four:
 * with one scale vector for A and B (sigma = tau) the sum moves into the residue domain,
 * C+ = A+ B-^T + B+ A-^T (mod m_j) and C- = C+^T.  A, B: n x k complex128 (lda, ldb >= n).  Lower triangle of C as for
 * zherk2m. */
int zher2k2m(int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc, int nmod,
             void* stream);

/* Real symmetric rank-k update C = A A^T (Section 5, SYRK) as the real part of the HERK of Z = A1 + i A2, where A1, A2 are
 * the two halves of the k dimension (a zero column is appended when k is odd): one real int8 GEMM of half the inner
 * dimension per modulus.  A: n x k real doubles (lda >= n); C: n x n real doubles (ldc >= n), lower triangle written. */
int dsyrk2m(int64_t n, int64_t k, const double* A, int64_t lda, double* C, int64_t ldc, int nmod, void* stream);

/* Real symmetric rank-2k update C = A B^T + B A^T (Section 5, SYR2K) as the real part of the HER2K of Z_A = A1 + i A2 and
 * Z_B = B1 + i B2.  A, B: n x k real doubles; C as for dsyrk2m. */
int dsyr2k2m(int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc, int nmod,
             void* stream);

/* (The paper has no counterpart for this entry point; it exists for deployment reasons only.)
 * Scale exponents without any allocation.  Some programs that would like to use this library are not allowed to
 * allocate device memory at the point of the call: a plug-in running inside a host application that handed the whole
 * GPU to its own memory pool at start-up, a service with a fixed memory budget that forbids cudaMalloc after
 * initialisation, or code on a latency-critical path where an allocation's implicit synchronisation is unacceptable.
 * They cannot provide the workspace the other entry points need.  This call computes, for the rows of A (m x k
 * complex128, column-major, lda >= m, device pointer), exactly the scale exponents e_i (sigma_i = 2^e_i, Algorithm 1
 * step 2) that zgemm2m(m, *, k, ..., nmod) uses under its default scaling rule (the rule of gemm2m_set_scaling(0), whatever
 * rule is selected at the time of the call), and writes them to e (int32[m], device pointer), using a scratch array
 * that is built into the library instead of a workspace.  It calls no cudaMalloc/cudaFree and no allocating library.
 * Returns GEMM2M_ERR_ARCH on a device that is not compute capability 10.0.
 *   - At most GEMM2M_STATIC_MAX_ROWS rows; more returns GEMM2M_ERR_WORKSPACE and launches nothing.
 *   - The built-in scratch (8 bytes per row of the maximum, 512 KB) is held by every GPU that loads the library until the
 *     process exits, is shared by all calls and keeps the last call's contents; the call clears what it uses.  Two calls
 *     that overlap on the same GPU (different streams) race on it: order them.
 *   - The first call on each device looks up the scratch's device address (with that device current).  Make that first
 *     call before starting any stream capture.
 *   - gemm2m_last_cuda_error is not updated by this entry point. */
#define GEMM2M_STATIC_MAX_ROWS 65536
int gemm2m_zscale_exponents_static(int64_t m, int64_t k, const double* A, int64_t lda, int nmod, int32_t* e, void* stream);

/* Waits for `stream` and returns GEMM2M_ERR_DEVICE_TIMEOUT if a kernel of an earlier call on the registered
 * workspace gave up a bounded wait (its results are then invalid), GEMM2M_ERR_CUDA on a CUDA error, else OK. */
int gemm2m_device_status(void* stream);

/* ---- instrumentation (used by the tests and the benchmark; not needed for normal use) ---- */

/* Phase timing: when enabled, every call records CUDA events around its phases on the call's stream (up to the 64 most
 * recent calls are kept).  Switching it on or off forgets earlier records. */
int gemm2m_set_profiling(int enabled);
/* Waits for the recorded calls and returns the average milliseconds per call of each phase: ms[0] = exponent scan,
 * ms[1] = quantise + residues (Eq. 2a), ms[2] = int8 GEMMs (Eq. 2b), ms[3] = post-processing (Eq. 2c + CRT + unscale);
 * *calls = number of calls averaged.  Each figure is the sum of the durations of the phase's kernels on the stream they run
 * on; with gemm2m_debug_set_overlap(1) zgemm2m/cgemm2m post-process one column panel on an internal stream while the next
 * panel's GEMMs run, and the four figures can then add up to more than the duration of the call.  The events between the
 * phases cost a few microseconds per call.  Host pointers; GEMM2M_ERR_ARG if nothing was recorded. */
int gemm2m_phase_ms(float ms[4], int* calls);
/* Number of kernels the last call launched (per phase in the same order, host pointer, may be NULL); returns total. */
int gemm2m_last_launch_count(int per_phase[4]);

/* Where the intermediate stages of a call live inside the workspace (byte offsets from its start), so that tests
 * can compare each stage with the CPU oracle.  Planes are indexed p = sign * nmod + j with sign 0 for "+", 1 for "-". */
typedef struct {
    int64_t off_exp_a;     /* int32[m]: scale exponents e_i, sigma_i = 2^e_i (rows of A)                 */
    int64_t off_exp_b;     /* int32[n]: scale exponents f_j, tau_j = 2^f_j (columns of B); HERK: unused  */
    int64_t off_apm;       /* int8 [2 nmod][m][kp]: residues of A, K contiguous                           */
    int64_t off_bpm;       /* int8 [2 nmod][n][kp]: residues of B, K contiguous; HERK: unused             */
    int64_t off_cpm;       /* int8 [2 nmod][n][ldp]: C+- mod m_j, M contiguous; HERK: [nmod][n][ldp], C+ only */
    int64_t kp;            /* padded K (multiple of 128; padding is zero)                                  */
    int64_t ldp;           /* leading dimension of the C+- planes (multiple of 16)                         */
    int64_t total_bytes;
} gemm2m_layout;
int gemm2m_workspace_layout(int op, int64_t m, int64_t n, int64_t k, int nmod, gemm2m_layout* out);

/* Failure handling, exercised without a fault: enqueues a one-thread kernel that waits, with the bounded wait every role of the
 * GEMM kernel uses, on a barrier nobody ever arrives on.  After budget_ns (checked about every 0.2 ms) the wait gives up, records
 * its code in the workspace's status word and the kernel returns; gemm2m_device_status() then reports
 * GEMM2M_ERR_DEVICE_TIMEOUT once and clears the word.  Needs a registered workspace (GEMM2M_ERR_WORKSPACE otherwise). */
int gemm2m_debug_wait_selftest(uint64_t budget_ns, void* stream);
/* Which int8 GEMM kernel later calls use: 0 = the tcgen05 kernel on CTA pairs (default), 1 = a plain CUDA-core check
 * kernel kept only so that tests can tell a fault in the tensor-core kernel from one in the pre/post kernels. */
int gemm2m_debug_set_gemm_kernel(int which);
/* Largest number of panels the output is cut into (default 8; panels are about 1024 to 2048 columns wide; the GEMMs of a panel
 * are one launch, its post-processing the next). */
int gemm2m_debug_set_panels(int max_panels);
/* 0 (default): every kernel of a call runs on the caller's stream, in order.  1: the post-processing of a panel (and, for
 * large operands, the exponent scan of B) runs on a library-owned stream beside the next panel's GEMMs, forked from and joined
 * back into the caller's stream with events.  Kept for measurement: on a GPU whose GEMM phase is power-limited it gains 1 to 3 % of a call. */
int gemm2m_debug_set_overlap(int enabled);
/* 1 (default): the residue, GEMM and post-processing kernels of a call are launched as programmatic dependents of the kernel
 * before them on the stream: a kernel may become resident while its predecessor drains, and waits on the device for the
 * predecessor's completion before it touches global memory, so results and ordering are those of plain launches.  0: plain
 * launches.  Kept for measurement (it matters for small problems, where launch latency is a visible share of a call). */
int gemm2m_debug_set_chained_launch(int enabled);

/* Host-only: copies the constants the library uses for `nmod` moduli and inner dimension k into caller arrays (host
 * pointers, any may be NULL), so that CPU tests can check them against an independent computation:
 *   scale[4]        = P_t, P_A, P_B, c_k of the scaling rule (herk != 0: P_A = P_B)
 *   crt_gr/gi[nmod*5] = signed base-2^40 digits of the folded CRT weights (real / imaginary part), crt_m[5] = digits of M
 *   nchunks         = number of digits in use
 *   res_w[nmod*16]  = int8 byte weights of the residue kernels: 8 for the real part, then 8 for the imaginary part */
int gemm2m_debug_tables(int nmod, int64_t k, int herk, int* scale, double* crt_gr, double* crt_gi, double* crt_m, int* nchunks,
                        int8_t* res_w);

/* Constants of the residue kernels' reduction modulo m_j (tests only; host pointers, nmod entries each, any may be NULL):
 *   y0_bits  = bit pattern of the float Y0 at which the real part's byte-weight sum starts
 *   cq       = the FMA addend 1.5 2^23 - Y0/m_j
 *   inv_m    = the float reciprocal in use
 *   xmax     = bound on the magnitude of the reduced sums
 *   margin   = (1/(2 m_j)) / ((Y0 + xmax) |inv_m - 1/m_j|): the quotient estimate is exact while this exceeds 1 */
/* The same constants for the real scheme of dgemm_ozaki2 (tests only; host pointers, any may be NULL): moduli[nmod],
 * scale[4] = P_t, P_A, P_B, c_k, crt_g[nmod*5] = digits of sym(q_j)(M/m_j), crt_m[5], nchunks, and the reduction constants. */
int gemm2m_debug_tables_real(int nmod, int64_t k, int* moduli, int* scale, double* crt_g, double* crt_m, int* nchunks, int32_t* y0_bits, float* cq,
                             float* inv_m, int32_t* xmax, double* margin);
int gemm2m_debug_residue_reduction(int nmod, int32_t* y0_bits, float* cq, float* inv_m, int32_t* xmax, double* margin);
/* Operand of the tensor-core contraction in the post-processing (tests only; host pointers, any may be NULL; variant 0 = the
 * complex GEMMs, 1 = the Eisenstein set, 2 = the rank-k family, whose planes are the C+ planes read directly, in K slots
 * 0 .. nmod-1, and mirrored, in slots H .. H+nmod-1 with H = nmod rounded up to 16).  Eq. (2c) (Eq. (1) for a 3M modulus) and the CRT of Section 3.1 are folded
 * into one weight per residue plane and part (real, imaginary), reduced to [0, M) and written in bytes:
 *   dims[3]   = residue planes, K-steps of 32 planes, chunks of four bytes (nb)
 *   digits    = [2][planes][24] bytes, least significant first: weight of the plane in the real / imaginary part
 *   consts[19]= M in base 2^32 (6 numbers, each times its power of 2^32; lower digits balanced), then per part the 6 numbers
 *               (1.5 2^52 + digit k of 128 x the sum of the part's weights) 2^(32k), then 1/M. */
int gemm2m_debug_post_operands(int variant, int nmod, uint8_t* digits, int* dims, double* consts);
/* The same for the Eisenstein set (tests only): scale[4], crt_gr / crt_gi[nmod*5] = digits of sym(4^-1 q_j)(M/m_j) and of
 * sym(-(4 d_j)^-1 q_j)(M/m_j), crt_m[5], nchunks, and the reduction constants. */
int gemm2m_debug_tables_eisenstein(int nmod, int64_t k, int* scale, double* crt_gr, double* crt_gi, double* crt_m, int* nchunks,
                                   int32_t* y0_bits, float* cq, float* inv_m, int32_t* xmax, double* margin);

#ifdef __cplusplus
}
#endif
#endif /* GEMM2M_H */

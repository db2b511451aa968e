// C-ABI entry points of the gemm2m library (declared in include/gemm2m.h): argument checks, workspace
// carving and the launch sequence of Algorithm 1.  Host code only enqueues; nothing here allocates device memory.
#include "../../include/gemm2m.h"

#include "common.cuh"

#include <cstdio>
#include <cstring>
#include <mutex>

using namespace gemm2m;

namespace {

// Per-device part of the library state: the registered workspace, the side stream with its ordering events, and what was
// learnt about the device.
constexpr int kHostPanels = 32;   // most column panels of a zgemm2m_host call

struct DevState {
    void* ws = nullptr;
    size_t ws_bytes = 0;
    cudaStream_t side = nullptr;  // library-owned stream on which the post-processing of a column panel overlaps the next panel's GEMMs
    cudaEvent_t panel_done[8] = {};
    cudaEvent_t side_done = nullptr;
    // zgemm2m_host: one stream per copy direction, and the events that order copies and kernels
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t call_begin = nullptr, a_ready = nullptr, b_ready[kHostPanels] = {}, g_ready[kHostPanels] = {}, c_ready[kHostPanels] = {}, c_done = nullptr;
    int sm_count = 0;
    int arch_ok = -1;
    int frags_key = 0;            // which post-processing operand the workspace holds: 0 = none, else 1 + nmod (+ 64 for the Eisenstein set)
};

struct State {
    std::mutex mu;
    DevState dev[kMaxDevices];
    int cur = 0;                  // device of the call being served (set by use_current_device)
    int profiling = 0;
    static constexpr int kProfSlots = 64, kMaxIntervals = 4 + 4 * kHostPanels, kMaxPanels = 8;
    struct Interval { cudaEvent_t a = nullptr, b = nullptr; int phase = 0; };
    struct Slot { Interval iv[kMaxIntervals]; int n = 0; };
    Slot slots[kProfSlots];       // timed intervals (phase, start, end) of the profiled calls
    int prof_calls = 0;           // profiled calls since profiling was switched on (each uses slot prof_calls % kProfSlots)
    Slot* cur_slot = nullptr;     // slot of the call being enqueued
    int max_panels = 8;           // most column panels per zgemm2m/cgemm2m call
    int chained = 1;              // 1 = the residue, GEMM and post-processing kernels are launched as programmatic dependents
    int overlap = 0;              // 1 = post-processing of a panel (and the scan of B) on the library's stream beside the next kernels
    int launches[4] = {0, 0, 0, 0};
    int gemm_kernel = 0;          // 0 = tcgen05 CTA pairs, 1 = check kernel
    int scaling = 0;              // 0 = largest part times sqrt(2k), 1 = 2-norm rule (zgemm2m / cgemm2m)
};
State g;
}  // namespace
bool gemm2m::chained_launch_enabled() { return g.chained != 0; }   // read while a call holds the library mutex
namespace {
DevState& D() { return g.dev[g.cur]; }
thread_local char g_cuda_err[256] = "no error";

int cuda_fail(cudaError_t e) {
    std::snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return GEMM2M_ERR_CUDA;
}
#define CK(expr)                                       \
    do {                                               \
        cudaError_t _e = (expr);                       \
        if (_e != cudaSuccess) return cuda_fail(_e);   \
    } while (0)

inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// Points D() at the state of the calling thread's current device (the caller holds g.mu).
void select_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) g.cur = dev;
}

// The same, and checks the device's architecture once.
int check_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GEMM2M_ERR_CUDA;
    g.cur = dev;
    if (D().arch_ok < 0) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return GEMM2M_ERR_CUDA;
        D().arch_ok = (prop.major == 10 && prop.minor == 0) ? 1 : 0;
        D().sm_count = prop.multiProcessorCount;
    }
    return D().arch_ok ? GEMM2M_OK : GEMM2M_ERR_ARCH;
}

// Workspace: [status 256 B][post-processing operand 3 KB][absmax A u64][absmax B u64][sumsq A u64][sumsq B u64][exp A i32][exp B i32][Apm][Bpm][Cpm], each
// 256-byte aligned.
struct Carve {
    int64_t off_status, off_frags, off_abs_a, off_abs_b, off_q_a, off_q_b, off_exp_a, off_exp_b, off_pack_a, off_pack_b, off_apm, off_bpm, off_cpm, kp, ldp, total;
    int64_t off_dev_a, off_dev_b, off_dev_c;      // zgemm2m_host: device copies of A (m x k), B (k x n) and C (m x n), compact
};

bool carve(int op, int64_t m, int64_t n, int64_t k, int nmod, Carve* c) {
    if (m < 0 || n < 0 || k < 0 || nmod < 1 || nmod > kMaxMod) return false;
    if (op < GEMM2M_OP_GAUSSIAN_INT || op > GEMM2M_OP_ZGEMM_HOST) return false;
    const bool host = op == GEMM2M_OP_ZGEMM_HOST;                               // zgemm2m plus device copies of the operands
    if (host) op = GEMM2M_OP_ZGEMM;
    const bool eis = op == GEMM2M_OP_ZGEMM_EISENSTEIN;                          // two planes per modulus of the Eisenstein set
    if (eis && nmod > kMaxEis) return false;
    const bool real_scheme = op == GEMM2M_OP_DGEMM_OZAKI2;                      // one plane per modulus of the real set
    if (real_scheme && nmod > kMaxReal) return false;
    const bool herk = op >= GEMM2M_OP_ZHERK && op <= GEMM2M_OP_DSYR2K;         // the rank-k family: one scale vector, C+ only
    const bool two = op == GEMM2M_OP_ZHER2K || op == GEMM2M_OP_DSYR2K;         // rank-2k: two operands
    const bool real_in = op == GEMM2M_OP_DSYRK || op == GEMM2M_OP_DSYR2K;      // real input, packed as Z = X1 + i X2
    if (herk && nmod > kMax2M) return false;                                   // the hybrid moduli serve the complex GEMMs only
    if (herk) m = n;
    if (real_in) k = (k + 1) / 2;
    const int64_t kp = round_up(k > 0 ? k : 1, 128), ldp = round_up(m > 0 ? m : 1, 16);
    int64_t off = 0;
    auto take = [&](int64_t bytes) { int64_t o = off; off = round_up(off + bytes, 256); return o; };
    c->off_status = take(256);
    c->off_frags = take(4 * kPostFragWords);    // tensor-core operand of the complex GEMMs' post-processing (digits of the CRT weights)
    c->off_abs_a = take(8 * m);
    c->off_abs_b = take(herk ? 0 : 8 * n);
    c->off_q_a = take(herk ? 0 : 8 * m);        // sums of squares of the 2-norm scaling rule (zeroed together with the maxima)
    c->off_q_b = take(herk ? 0 : 8 * n);
    c->off_exp_a = take(4 * m);
    c->off_exp_b = take(herk ? 0 : 4 * n);
    c->off_pack_a = take(real_in ? 16 * n * k : 0);
    c->off_pack_b = take(real_in && two ? 16 * n * k : 0);
    const int64_t planes = real_scheme ? nmod : eis ? 2 * nmod : plane_count(nmod);   // 2 per 2M modulus, 3 per 3M modulus
    c->off_apm = take(planes * m * kp);
    c->off_bpm = take((herk && !two) ? 0 : planes * n * kp);
    c->off_cpm = take((herk ? (int64_t)nmod : planes) * n * ldp);
    c->off_dev_a = take(host ? 16 * m * k : 0);
    c->off_dev_b = take(host ? 16 * k * n : 0);
    c->off_dev_c = take(host ? 16 * m * n : 0);
    c->kp = kp;
    c->ldp = ldp;
    c->total = off;
    return true;
}

struct Phases {   // event bookkeeping of one call: every phase is a set of intervals, each on the stream its kernels run on
    bool on = false;
    cudaError_t begin(int phase, cudaStream_t st) {
        if (!on || g.cur_slot->n >= State::kMaxIntervals) return cudaSuccess;
        State::Interval& iv = g.cur_slot->iv[g.cur_slot->n];
        iv.phase = phase;
        if (!iv.a) { cudaError_t e = cudaEventCreate(&iv.a); if (e != cudaSuccess) return e; }
        if (!iv.b) { cudaError_t e = cudaEventCreate(&iv.b); if (e != cudaSuccess) return e; }
        return cudaEventRecord(iv.a, st);
    }
    cudaError_t end(cudaStream_t st) {
        if (!on || g.cur_slot->n >= State::kMaxIntervals) return cudaSuccess;
        return cudaEventRecord(g.cur_slot->iv[g.cur_slot->n++].b, st);
    }
    void done() { if (on) ++g.prof_calls; }
};

int begin_call(Phases* ph) {
    ph->on = g.profiling != 0;
    std::memset(g.launches, 0, sizeof(g.launches));
    if (ph->on) {
        g.cur_slot = &g.slots[g.prof_calls % State::kProfSlots];
        g.cur_slot->n = 0;
    }
    return GEMM2M_OK;
}

// Side stream and ordering events, created on first use (no device memory involved).
int ensure_side_stream() {
    if (!D().side) CK(cudaStreamCreateWithFlags(&D().side, cudaStreamNonBlocking));
    for (auto& e : D().panel_done)
        if (!e) CK(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    if (!D().side_done) CK(cudaEventCreateWithFlags(&D().side_done, cudaEventDisableTiming));
    return GEMM2M_OK;
}

int ensure_copy_streams() {
    if (!D().h2d) CK(cudaStreamCreateWithFlags(&D().h2d, cudaStreamNonBlocking));
    if (!D().d2h) CK(cudaStreamCreateWithFlags(&D().d2h, cudaStreamNonBlocking));
    auto make = [](cudaEvent_t& e) { return e ? cudaSuccess : cudaEventCreateWithFlags(&e, cudaEventDisableTiming); };
    CK(make(D().call_begin));
    CK(make(D().a_ready));
    CK(make(D().c_done));
    for (auto& e : D().b_ready) CK(make(e));
    for (auto& e : D().g_ready) CK(make(e));
    for (auto& e : D().c_ready) CK(make(e));
    return GEMM2M_OK;
}

constexpr int64_t kMaxRows = 65535LL * 32;   // grid.y limit of the residue kernels

// hex: the Eisenstein variant's lattice rounding in front of the same residue arithmetic (complex double only).
template <typename T>
int run_residues(const T* X, int64_t ld, bool k_contiguous, bool conj, int64_t R, int64_t K, int64_t Kp, int32_t* e,
                 const ResidueTable& tab, int width, int8_t* planes, int* dev_status, cudaStream_t st, bool hex = false,
                 ScaleFrom from = ScaleFrom()) {
    if (hex) {
        if constexpr (sizeof(T) == 8) {
            CK(launch_residues_hex(X, ld, k_contiguous, conj, R, K, Kp, e, tab, width == 1, planes, st, &g.launches[1], from));
            return GEMM2M_OK;
        } else {
            return GEMM2M_ERR_ARG;
        }
    }
    (void)dev_status;
    CK(launch_residues_fp<T>(X, ld, k_contiguous, conj, R, K, Kp, e, tab, width, planes, st, &g.launches[1], 0, from));
    return GEMM2M_OK;
}

int run_gemm(const GemmArgs& a, int64_t klim, cudaStream_t st) {
    if (g.gemm_kernel == 1) CK(launch_gemm_check(a, klim, st, &g.launches[2]));
    else CK(launch_gemm_tcgen05_pair(a, klim, D().sm_count, st, &g.launches[2]));
    return GEMM2M_OK;
}

// Panel loop shared by every entry point: the rows [0, n) of the GEMM's row operand (columns of C for the GEMMs, rows of the
// lower triangle for the rank-k family) are cut into panels of about 1024 rows up to four of them, then of about 2048 rows
// (more, narrower panels also keep the operand slices of a launch inside the L2: 16384 columns in 8 panels measured 6-8 %
// faster than in 4).  gemm(r0, r1) enqueues the GEMMs of a panel on the caller's stream; post(r0, r1, stream) its
// post-processing, by default on the same stream right behind them.  With the overlap switched on (gemm2m_debug_set_overlap)
// the post-processing of every panel but the last runs on the library's stream beside the GEMMs of the next panel, and the
// call is complete on the caller's stream only when the library's stream has been joined back.  Measured with whole calls of
// the two modes alternating in one loop, the overlap gains 0.4 % at 8192^3 and loses 0.8 % for cgemm2m at 16384 x 16384 x
// 4096: the GEMM phase runs at the board's power limit, and what runs beside it slows it down by what it hides.
// (Panel count at 8192 columns, 30 back-to-back calls each: 1 panel 17.4-17.7 ms, 2 panels 17.2-17.4, 4 panels 15.7-16.3,
// 8 panels 16.5-16.7: fewer launches would read the planes of A less often, but the short post-processing launches between the
// GEMM launches let the power-limited clock recover, which is worth more.)
template <typename GemmFn, typename PostFn>
int panel_pipeline(int64_t n, cudaStream_t st, Phases& ph, GemmFn gemm, PostFn post) {
    int panels = (int)(n / 1024);
    if (panels > 4) panels = (int)(n / 2048) > 4 ? (int)(n / 2048) : 4;
    panels = panels < 1 ? 1 : (panels > g.max_panels ? g.max_panels : panels);
    const int64_t panel_rows = round_up((n + panels - 1) / panels, 256);
    const bool overlap = g.overlap && panels > 1;
    if (overlap) { if (int s = ensure_side_stream()) return s; }
    for (int pnl = 0; pnl < panels; ++pnl) {
        const int64_t r0 = pnl * panel_rows, r1 = (r0 + panel_rows < n) ? r0 + panel_rows : n;
        if (r0 >= r1) break;
        CK(ph.begin(2, st));
        if (int s = gemm(r0, r1)) return s;
        CK(ph.end(st));
        const bool last = r1 >= n || !overlap;
        cudaStream_t ps = last ? st : D().side;
        if (!last) {
            CK(cudaEventRecord(D().panel_done[pnl], st));
            CK(cudaStreamWaitEvent(D().side, D().panel_done[pnl], 0));
        }
        CK(ph.begin(3, ps));
        CK(post(r0, r1, ps));
        CK(ph.end(ps));
    }
    if (overlap) {
        CK(cudaEventRecord(D().side_done, D().side));
        CK(cudaStreamWaitEvent(st, D().side_done, 0));
    }
    return GEMM2M_OK;
}

// transa / transb: 'N' (as stored), 'T' (transposed) or 'C' (conjugate transposed) operand, BLAS style; alpha, beta: host
// pointers to (re, im) pairs or null for 1 and 0.  C = alpha op(A) op(B) + beta C with op(A) m x k and op(B) k x n.
template <typename T>
int xgemm2m(int op, char transa, char transb, int64_t m, int64_t n, int64_t k, const double* alpha, const T* A, int64_t lda, const T* B,
            int64_t ldb, const double* beta, T* C, int64_t ldc, int nmod, void* stream) {
    std::lock_guard<std::mutex> lock(g.mu);
    auto norm = [](char c) { return (c == 'n' || c == 'N') ? 'N' : (c == 't' || c == 'T') ? 'T' : (c == 'c' || c == 'C') ? 'C' : '?'; };
    const char ta = norm(transa), tb = norm(transb);
    if (ta == '?' || tb == '?') return GEMM2M_ERR_ARG;
    if (m < 0 || n < 0 || k < 0) return GEMM2M_ERR_ARG;
    const int64_t rows_a = ta == 'N' ? m : k, rows_b = tb == 'N' ? k : n;      // rows of the matrices as stored
    if (lda < (rows_a > 1 ? rows_a : 1) || ldb < (rows_b > 1 ? rows_b : 1) || ldc < (m > 1 ? m : 1)) return GEMM2M_ERR_ARG;
    const bool eis = op == GEMM2M_OP_ZGEMM_EISENSTEIN;
    if (nmod < 1 || nmod > (eis ? kMaxEis : kMaxMod)) return GEMM2M_ERR_NMOD;
    if (m > kMaxRows || n > kMaxRows) return GEMM2M_ERR_ARG;
    if (m == 0 || n == 0) return GEMM2M_OK;
    const bool alpha_zero = alpha && alpha[0] == 0.0 && alpha[1] == 0.0;
    if (!C || (k > 0 && !alpha_zero && (!A || !B))) return GEMM2M_ERR_ARG;
    if (int s = check_device()) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if (k == 0 || alpha_zero) {          // nothing to multiply: C = beta C (A and B are not referenced)
        std::memset(g.launches, 0, sizeof(g.launches));
        if (!beta || (beta[0] == 0.0 && beta[1] == 0.0))
            CK(cudaMemset2DAsync(C, (size_t)ldc * 2 * sizeof(T), 0, (size_t)m * 2 * sizeof(T), (size_t)n, st));
        else if (!(beta[0] == 1.0 && beta[1] == 0.0))
            CK(launch_scale_c<T>(C, m, n, ldc, beta, st, &g.launches[3]));
        return GEMM2M_OK;
    }
    Carve c;
    if (!carve(op, m, n, k, nmod, &c)) return GEMM2M_ERR_ARG;
    if (!D().ws || D().ws_bytes < (size_t)c.total) return GEMM2M_ERR_WORKSPACE;
    char* ws = (char*)D().ws;
    int* dev_status = (int*)(ws + c.off_status);
    uint64_t* absA = (uint64_t*)(ws + c.off_abs_a);
    uint64_t* absB = (uint64_t*)(ws + c.off_abs_b);
    int32_t* eA = (int32_t*)(ws + c.off_exp_a);
    int32_t* eB = (int32_t*)(ws + c.off_exp_b);
    int8_t* apm = (int8_t*)(ws + c.off_apm);
    int8_t* bpm = (int8_t*)(ws + c.off_bpm);
    int8_t* cpm = (int8_t*)(ws + c.off_cpm);

    const ScaleTargets sc = eis ? scale_targets_eis(nmod, k) : scale_targets(nmod, k, false);
    if (eis && sc.PB - sc.ck < 2) return GEMM2M_ERR_NMOD;          // the lattice rounding needs scaled parts of 4 or more
    ResidueTable rtab;
    PostMmaTable ptab;
    if (eis) { build_residue_table_eis(nmod, &rtab); build_post_mma_table_eis(nmod, &ptab); }
    else { build_residue_table(nmod, &rtab); build_post_mma_table(nmod, &ptab); }
    uint32_t* frags = (uint32_t*)(ws + c.off_frags);
    // quantised parts stay below 2^(P - c_k) with the max-based rule and below 2^P with the 2-norm rule
    const bool two_norm_mode = !eis && g.scaling == 1 && k <= (1ll << 22);
    // (Eisenstein variant: the coordinate u reaches 2^(P - c_k + 1) + 1)
    const int head = eis ? 2 : 0;
    const bool wideA = two_norm_mode ? sc.PA > 61 : sc.PA - sc.ck + head > 62, wideB = two_norm_mode ? sc.PB > 61 : sc.PB - sc.ck + head > 62;
    // narrow: every quantised part stays below 2^30 in magnitude (the same bounds, 32 bits down), which halves the residue kernel's byte-weight chains
    const bool narrowA = !eis && (two_norm_mode ? sc.PA <= 29 : sc.PA - sc.ck + head <= 30), narrowB = !eis && (two_norm_mode ? sc.PB <= 29 : sc.PB - sc.ck + head <= 30);
    const int widthA = wideA ? 1 : narrowA ? 2 : 0, widthB = wideB ? 1 : narrowB ? 2 : 0;

    Phases ph;
    if (int s = begin_call(&ph)) return s;
    // step 2: scale factors.  Everything runs on the caller's stream, one phase after the other.  (With the overlap switched
    // on, the scan of B, bandwidth-bound, runs on the library's stream beside the scan and the residues of A, which are bound
    // by arithmetic, and the residues of B wait for it; not for small operands, whose scan is shorter than a fork and join.)
    const bool side_scan = g.overlap && k * n >= (1ll << 24);
    if (side_scan) { if (int s = ensure_side_stream()) return s; }
    cudaStream_t sb = side_scan ? D().side : st;
    CK(cudaMemsetAsync(ws + c.off_abs_a, 0, (size_t)(c.off_exp_a - c.off_abs_a), st));
    const int frags_key = 1 + nmod + (eis ? 64 : 0);           // the operand of the post-processing stays in the workspace between calls
    if (D().frags_key != frags_key) {
        CK(launch_post_operands(ptab, frags, st, &g.launches[3]));
        D().frags_key = frags_key;
    }
    if (sb != st) {
        CK(cudaEventRecord(D().panel_done[0], st));
        CK(cudaStreamWaitEvent(sb, D().panel_done[0], 0));
    }
    uint64_t* qA = (uint64_t*)(ws + c.off_q_a);
    uint64_t* qB = (uint64_t*)(ws + c.off_q_b);
    CK(ph.begin(0, sb));
    // columns of op(B) are columns of B as stored ('N') or its rows ('T', 'C')
    if (tb == 'N') CK(launch_scan_cols<T>(B, k, n, ldb, absB, sb, &g.launches[0]));
    else CK(launch_scan_rows<T>(B, n, k, ldb, absB, sb, &g.launches[0]));
    // (largest-part rule: the residue kernels form the exponents from the maxima themselves)
    if (!two_norm_mode) {}
    else if (tb == 'N') CK(launch_exponents_2norm<T>(B, k, n, ldb, false, absB, qB, sc.PB, eB, sb, &g.launches[0]));
    else CK(launch_exponents_2norm<T>(B, n, k, ldb, true, absB, qB, sc.PB, eB, sb, &g.launches[0]));
    CK(ph.end(sb));
    if (sb != st) CK(cudaEventRecord(D().side_done, sb));
    CK(ph.begin(0, st));
    // rows of op(A) are rows of A as stored ('N') or its columns ('T', 'C')
    const bool after_kernel = sb == st && !ph.on;          // directly behind the scan of B (no event in between)
    if (ta == 'N') CK(launch_scan_rows<T>(A, m, k, lda, absA, st, &g.launches[0], after_kernel));
    else CK(launch_scan_cols<T>(A, k, m, lda, absA, st, &g.launches[0], after_kernel));
    if (!two_norm_mode) {}                                                                          // (2-norm rule: not for k > 2^22,
    else if (ta == 'N') CK(launch_exponents_2norm<T>(A, m, k, lda, true, absA, qA, sc.PA, eA, st, &g.launches[0]));   // where the sums
    else CK(launch_exponents_2norm<T>(A, k, m, lda, false, absA, qA, sc.PA, eA, st, &g.launches[0]));   // of squares would not fit 64 bits)
    CK(ph.end(st));
    // step 3 + Eq. (2a)
    CK(ph.begin(1, st));
    ScaleFrom fromA, fromB;
    if (!two_norm_mode) {
        fromA.absmax = (const unsigned long long*)absA; fromA.P = sc.PA; fromA.ck = sc.ck;
        fromB.absmax = (const unsigned long long*)absB; fromB.P = sc.PB; fromB.ck = sc.ck;
    }
    if (int s = run_residues<T>(A, lda, ta != 'N', ta == 'C', m, k, c.kp, eA, rtab, widthA, apm, dev_status, st, eis, fromA)) return s;
    if (sb != st) CK(cudaStreamWaitEvent(st, D().side_done, 0));
    if (int s = run_residues<T>(B, ldb, tb == 'N', tb == 'C', n, k, c.kp, eB, rtab, widthB, bpm, dev_status, st, eis, fromB)) return s;
    CK(ph.end(st));
    // Eq. (2b): 2 real int8 GEMMs per 2M modulus (3 per 3M modulus of the hybrid, Eq. (1)); TMEM lanes = columns of C (rows of Bpm), TMEM columns = rows of C (rows of Apm).
    // The columns of C are cut into panels: one GEMM launch and one launch of Eq. (2c) + steps 5-7 per panel, in order.
    // (Forming the residues of B panel by panel too, each right before its panel's GEMMs, was measured and brought nothing:
    // 16.0-16.8 against 16.1-16.2 ms per call at 8192^3 in a long run.)
    GemmArgs ga;
    ga.rowop = bpm; ga.colop = apm;
    ga.R = n; ga.Cn = m; ga.Kp = c.kp;
    const int nplanes = eis ? 2 * nmod : plane_count(nmod);
    ga.row_planes = ga.col_planes = nplanes;
    ga.row_plane0 = ga.col_plane0 = 0;
    ga.nbatch = nplanes;
    ga.out = cpm; ga.ldp = c.ldp; ga.accumulate = 0;
    if (eis) build_mod_table_eis(nmod, &ga.mods);
    else build_mod_table(nmod, true, &ga.mods);
    ga.dev_status = dev_status;
    const int64_t klim = eis ? gemm_k_limit_eis() : gemm_k_limit(nmod);
    if (int s = panel_pipeline(n, st, ph,
            [&](int64_t j0, int64_t j1) { ga.row_begin = j0; ga.row_end = j1; return run_gemm(ga, klim, st); },
            [&](int64_t j0, int64_t j1, cudaStream_t ps) {
                return launch_post_fp<T>(cpm, c.ldp, m, n, j0, j1, eA, eB, ptab, frags, C, ldc, alpha, beta, ps, &g.launches[3]);
            })) return s;
    ph.done();
    return GEMM2M_OK;
}

// zgemm2m on HOST operands: the copies are part of the call and overlap its kernels.  A goes up first (every GEMM needs all
// of its planes); B goes up in column panels, and each panel is scanned, reduced to residues, multiplied and post-processed
// while the next one is still on the bus; the finished column panel of C goes down beside the next panel's work.  The
// copies run on two library-owned streams (one per direction), ordered against the caller's stream by events; the call is
// complete on the caller's stream when the last panel of C has arrived in host memory.
int zgemm_host(int64_t m, int64_t n, int64_t k, const double* hA, int64_t lda, const double* hB, int64_t ldb, double* hC, int64_t ldc,
               int nmod, void* stream) {
    std::lock_guard<std::mutex> lock(g.mu);
    if (m < 0 || n < 0 || k < 0) return GEMM2M_ERR_ARG;
    if (lda < (m > 1 ? m : 1) || ldb < (k > 1 ? k : 1) || ldc < (m > 1 ? m : 1)) return GEMM2M_ERR_ARG;
    if (nmod < 1 || nmod > kMaxMod) return GEMM2M_ERR_NMOD;
    if (m > kMaxRows || n > kMaxRows) return GEMM2M_ERR_ARG;
    if (m == 0 || n == 0) return GEMM2M_OK;
    if (!hC || (k > 0 && (!hA || !hB))) return GEMM2M_ERR_ARG;
    if (int s = check_device()) return s;
    cudaStream_t st = (cudaStream_t)stream;
    Carve c;
    if (!carve(GEMM2M_OP_ZGEMM_HOST, m, n, k, nmod, &c)) return GEMM2M_ERR_ARG;
    if (!D().ws || D().ws_bytes < (size_t)c.total) return GEMM2M_ERR_WORKSPACE;
    char* ws = (char*)D().ws;
    double* dA = (double*)(ws + c.off_dev_a);
    double* dB = (double*)(ws + c.off_dev_b);
    double* dC = (double*)(ws + c.off_dev_c);
    const size_t col_a = (size_t)m * 16, col_b = (size_t)k * 16;              // bytes of one column of A / C and of B
    std::memset(g.launches, 0, sizeof(g.launches));
    if (k == 0) {                                                              // C = 0
        CK(cudaMemsetAsync(dC, 0, col_a * (size_t)n, st));
        CK(cudaMemcpy2DAsync(hC, (size_t)ldc * 16, dC, col_a, col_a, (size_t)n, cudaMemcpyDeviceToHost, st));
        return GEMM2M_OK;
    }
    if (int s = ensure_side_stream()) return s;
    if (int s = ensure_copy_streams()) return s;
    int* dev_status = (int*)(ws + c.off_status);
    uint64_t* absA = (uint64_t*)(ws + c.off_abs_a);
    uint64_t* absB = (uint64_t*)(ws + c.off_abs_b);
    int32_t* eA = (int32_t*)(ws + c.off_exp_a);
    int32_t* eB = (int32_t*)(ws + c.off_exp_b);
    int8_t* apm = (int8_t*)(ws + c.off_apm);
    int8_t* bpm = (int8_t*)(ws + c.off_bpm);
    int8_t* cpm = (int8_t*)(ws + c.off_cpm);
    const ScaleTargets sc = scale_targets(nmod, k, false);
    ResidueTable rtab;
    PostMmaTable ptab;
    build_residue_table(nmod, &rtab);
    build_post_mma_table(nmod, &ptab);
    uint32_t* frags = (uint32_t*)(ws + c.off_frags);
    const bool wideA = sc.PA - sc.ck > 62, wideB = sc.PB - sc.ck > 62;
    Phases ph;
    if (int s = begin_call(&ph)) return s;

    // column panels of B and C: narrow, so that the last panel's kernels and download, which nothing hides, stay short
    // (the kernels hide behind the upload of B whatever the panel width; 256-column panels measured 43.4 ms per call at
    // 8192^3 against 44.4 ms with 512 and 45.3 ms with 1024 columns)
    int panels = (int)(n / 256);
    panels = panels < 1 ? 1 : (panels > kHostPanels ? kHostPanels : panels);
    const int64_t panel_cols = round_up((n + panels - 1) / panels, 256);

    // uploads: after everything the caller's stream holds so far (an earlier call may still read the device copies)
    cudaStream_t up = D().h2d, down = D().d2h, side = D().side;
    CK(cudaEventRecord(D().call_begin, st));
    CK(cudaStreamWaitEvent(up, D().call_begin, 0));
    CK(cudaMemcpy2DAsync(dA, col_a, hA, (size_t)lda * 16, col_a, (size_t)k, cudaMemcpyHostToDevice, up));
    CK(cudaEventRecord(D().a_ready, up));
    int used = 0;
    for (int p = 0; p < panels; ++p) {
        const int64_t j0 = p * panel_cols, j1 = (j0 + panel_cols < n && p + 1 < panels) ? j0 + panel_cols : n;
        if (j0 >= j1) break;
        CK(cudaMemcpy2DAsync(dB + 2 * j0 * k, col_b, hB + 2 * j0 * ldb, (size_t)ldb * 16, col_b, (size_t)(j1 - j0), cudaMemcpyHostToDevice, up));
        CK(cudaEventRecord(D().b_ready[p], up));
        used = p + 1;
    }
    // A: steps 2-4 as in zgemm2m
    CK(cudaMemsetAsync(ws + c.off_abs_a, 0, (size_t)(c.off_exp_a - c.off_abs_a), st));
    if (D().frags_key != 1 + nmod) {
        CK(launch_post_operands(ptab, frags, st, &g.launches[3]));
        D().frags_key = 1 + nmod;
    }
    CK(cudaStreamWaitEvent(st, D().a_ready, 0));
    CK(ph.begin(0, st));
    CK(launch_scan_rows<double>(dA, m, k, m, absA, st, &g.launches[0]));
    CK(launch_exponents<double>(absA, m, sc.PA, sc.ck, eA, st, &g.launches[0]));
    CK(ph.end(st));
    CK(ph.begin(1, st));
    CK(launch_residues_fp<double>(dA, m, false, false, m, k, c.kp, eA, rtab, wideA, apm, st, &g.launches[1]));
    CK(ph.end(st));
    GemmArgs ga;
    ga.rowop = bpm; ga.colop = apm;
    ga.R = n; ga.Cn = m; ga.Kp = c.kp;
    ga.row_planes = ga.col_planes = plane_count(nmod);
    ga.row_plane0 = ga.col_plane0 = 0;
    ga.nbatch = plane_count(nmod);
    ga.out = cpm; ga.ldp = c.ldp; ga.accumulate = 0;
    build_mod_table(nmod, true, &ga.mods);
    ga.dev_status = dev_status;
    for (int p = 0; p < used; ++p) {
        const int64_t j0 = p * panel_cols, j1 = (j0 + panel_cols < n && p + 1 < panels) ? j0 + panel_cols : n;
        const double* Bp = dB + 2 * j0 * k;
        // the scale factor of a column of B depends on that column alone: steps 2-4 of this panel's columns
        CK(cudaStreamWaitEvent(st, D().b_ready[p], 0));
        CK(ph.begin(0, st));
        CK(launch_scan_cols<double>(Bp, k, j1 - j0, k, absB + j0, st, &g.launches[0]));
        CK(launch_exponents<double>(absB + j0, j1 - j0, sc.PB, sc.ck, eB + j0, st, &g.launches[0]));
        CK(ph.end(st));
        CK(ph.begin(1, st));
        CK(launch_residues_fp<double>(Bp, k, true, false, j1 - j0, k, c.kp, eB + j0, rtab, wideB, bpm + j0 * c.kp, st, &g.launches[1], n));
        CK(ph.end(st));
        CK(ph.begin(2, st));
        ga.row_begin = j0; ga.row_end = j1;
        if (int s = run_gemm(ga, gemm_k_limit(nmod), st)) return s;
        CK(ph.end(st));
        // Eq. (2c) + steps 5-7 of the panel on the side stream, then its columns of C go down
        CK(cudaEventRecord(D().g_ready[p], st));
        CK(cudaStreamWaitEvent(side, D().g_ready[p], 0));
        CK(ph.begin(3, side));
        CK(launch_post_fp<double>(cpm, c.ldp, m, n, j0, j1, eA, eB, ptab, frags, dC, m, nullptr, nullptr, side, &g.launches[3]));
        CK(ph.end(side));
        CK(cudaEventRecord(D().c_ready[p], side));
        CK(cudaStreamWaitEvent(down, D().c_ready[p], 0));
        CK(cudaMemcpy2DAsync(hC + 2 * j0 * ldc, (size_t)ldc * 16, dC + 2 * j0 * m, col_a, col_a, (size_t)(j1 - j0), cudaMemcpyDeviceToHost, down));
    }
    CK(cudaEventRecord(D().c_done, down));
    CK(cudaStreamWaitEvent(st, D().c_done, 0));
    ph.done();
    return GEMM2M_OK;
}

}  // namespace

extern "C" {

const char* gemm2m_status_string(int status) {
    switch (status) {
        case GEMM2M_OK: return "GEMM2M_OK";
        case GEMM2M_ERR_ARG: return "GEMM2M_ERR_ARG";
        case GEMM2M_ERR_NMOD: return "GEMM2M_ERR_NMOD";
        case GEMM2M_ERR_WORKSPACE: return "GEMM2M_ERR_WORKSPACE";
        case GEMM2M_ERR_CUDA: return "GEMM2M_ERR_CUDA";
        case GEMM2M_ERR_ARCH: return "GEMM2M_ERR_ARCH";
        case GEMM2M_ERR_DEVICE_TIMEOUT: return "GEMM2M_ERR_DEVICE_TIMEOUT";
        default: return "GEMM2M_UNKNOWN";
    }
}

const char* gemm2m_last_cuda_error(void) { return g_cuda_err; }

int gemm2m_max_moduli(void) { return kMaxMod; }

int gemm2m_max_2m_moduli(void) { return kMax2M; }

int gemm2m_modulus(int j, int* m, int* s) {
    if (j < 0 || j >= kMaxMod) return GEMM2M_ERR_ARG;
    if (m) *m = modulus_value(j);
    if (s) *s = modulus_root(j);
    return GEMM2M_OK;
}

size_t gemm2m_workspace_bytes(int op, int64_t m, int64_t n, int64_t k, int nmod) {
    Carve c;
    if (op == GEMM2M_OP_GAUSSIAN_INT && nmod > 8) return 0;
    if (!carve(op, m, n, k, nmod, &c)) return 0;
    return (size_t)c.total;
}

int gemm2m_workspace_layout(int op, int64_t m, int64_t n, int64_t k, int nmod, gemm2m_layout* out) {
    Carve c;
    if (!out || !carve(op, m, n, k, nmod, &c)) return GEMM2M_ERR_ARG;
    out->off_exp_a = c.off_exp_a;
    out->off_exp_b = c.off_exp_b;
    out->off_apm = c.off_apm;
    out->off_bpm = c.off_bpm;
    out->off_cpm = c.off_cpm;
    out->kp = c.kp;
    out->ldp = c.ldp;
    out->total_bytes = c.total;
    return GEMM2M_OK;
}

int gemm2m_set_workspace(void* dev_ptr, size_t bytes) {
    std::lock_guard<std::mutex> lock(g.mu);
    if ((dev_ptr == nullptr) != (bytes == 0)) return GEMM2M_ERR_ARG;
    if (((uintptr_t)dev_ptr & 255) != 0) return GEMM2M_ERR_ARG;
    select_device();
    D().ws = dev_ptr;
    D().ws_bytes = bytes;
    D().frags_key = 0;
    if (dev_ptr) CK(cudaMemset(dev_ptr, 0, 256));   // device status word
    return GEMM2M_OK;
}

int gemm2m_gaussian_int(int64_t m, int64_t n, int64_t k, const int8_t* Ar, const int8_t* Ai, int64_t lda, const int8_t* Br,
                        const int8_t* Bi, int64_t ldb, int64_t* Cr, int64_t* Ci, int64_t ldc, int nmod, void* stream) {
    std::lock_guard<std::mutex> lock(g.mu);
    if (m < 0 || n < 0 || k < 0) return GEMM2M_ERR_ARG;
    if (lda < (m > 1 ? m : 1) || ldb < (k > 1 ? k : 1) || ldc < (m > 1 ? m : 1)) return GEMM2M_ERR_ARG;
    if (nmod < 1 || nmod > 8) return GEMM2M_ERR_NMOD;
    if (m > kMaxRows || n > kMaxRows) return GEMM2M_ERR_ARG;
    if (m == 0 || n == 0) return GEMM2M_OK;
    if (!Cr || !Ci || (k > 0 && (!Ar || !Ai || !Br || !Bi))) return GEMM2M_ERR_ARG;
    if (int s = check_device()) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if (k == 0) {
        CK(cudaMemset2DAsync(Cr, (size_t)ldc * 8, 0, (size_t)m * 8, (size_t)n, st));
        CK(cudaMemset2DAsync(Ci, (size_t)ldc * 8, 0, (size_t)m * 8, (size_t)n, st));
        return GEMM2M_OK;
    }
    Carve c;
    if (!carve(GEMM2M_OP_GAUSSIAN_INT, m, n, k, nmod, &c)) return GEMM2M_ERR_ARG;
    if (!D().ws || D().ws_bytes < (size_t)c.total) return GEMM2M_ERR_WORKSPACE;
    char* ws = (char*)D().ws;
    int8_t* apm = (int8_t*)(ws + c.off_apm);
    int8_t* bpm = (int8_t*)(ws + c.off_bpm);
    int8_t* cpm = (int8_t*)(ws + c.off_cpm);
    ResidueTable rtab;
    build_residue_table(nmod, &rtab);
    CrtTableInt ctab;
    build_crt_table_int(nmod, &ctab);
    Phases ph;
    if (int s = begin_call(&ph)) return s;
    CK(ph.begin(1, st));
    CK(launch_residues_int8(Ar, Ai, lda, false, m, k, c.kp, rtab, apm, st, &g.launches[1]));
    CK(launch_residues_int8(Br, Bi, ldb, true, n, k, c.kp, rtab, bpm, st, &g.launches[1]));
    CK(ph.end(st));
    GemmArgs ga;
    ga.rowop = bpm; ga.colop = apm;
    ga.R = n; ga.Cn = m; ga.Kp = c.kp;
    ga.row_planes = ga.col_planes = 2 * nmod;
    ga.row_plane0 = ga.col_plane0 = 0;
    ga.nbatch = 2 * nmod;
    ga.out = cpm; ga.ldp = c.ldp; ga.accumulate = 0;
    build_mod_table(nmod, true, &ga.mods);
    ga.dev_status = (int*)(ws + c.off_status);
    ga.row_begin = 0; ga.row_end = n;
    CK(ph.begin(2, st));
    if (int s = run_gemm(ga, gemm_k_limit(nmod), st)) return s;
    CK(ph.end(st));
    CK(ph.begin(3, st));
    CK(launch_post_int(cpm, c.ldp, m, n, ctab, Cr, Ci, ldc, st, &g.launches[3]));
    CK(ph.end(st));
    ph.done();
    return GEMM2M_OK;
}

int zgemm2m(int64_t m, int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc,
            int nmod, void* stream) {
    return xgemm2m<double>(GEMM2M_OP_ZGEMM, 'N', 'N', m, n, k, nullptr, A, lda, B, ldb, nullptr, C, ldc, nmod, stream);
}

int zgemm2m_host(int64_t m, int64_t n, int64_t k, const double* A_host, int64_t lda, const double* B_host, int64_t ldb, double* C_host,
                 int64_t ldc, int nmod, void* stream) {
    return zgemm_host(m, n, k, A_host, lda, B_host, ldb, C_host, ldc, nmod, stream);
}

int cgemm2m(int64_t m, int64_t n, int64_t k, const float* A, int64_t lda, const float* B, int64_t ldb, float* C, int64_t ldc, int nmod,
            void* stream) {
    return xgemm2m<float>(GEMM2M_OP_CGEMM, 'N', 'N', m, n, k, nullptr, A, lda, B, ldb, nullptr, C, ldc, nmod, stream);
}

int zgemm2m_eisenstein(int64_t m, int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc,
                       int nmod, void* stream) {
    return xgemm2m<double>(GEMM2M_OP_ZGEMM_EISENSTEIN, 'N', 'N', m, n, k, nullptr, A, lda, B, ldb, nullptr, C, ldc, nmod, stream);
}

int zgemm2m_eisenstein_ex(char transa, char transb, int64_t m, int64_t n, int64_t k, const double* alpha, const double* A, int64_t lda,
                          const double* B, int64_t ldb, const double* beta, double* C, int64_t ldc, int nmod, void* stream) {
    return xgemm2m<double>(GEMM2M_OP_ZGEMM_EISENSTEIN, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, nmod, stream);
}

int gemm2m_max_eisenstein_moduli(void) { return kMaxEis; }

int gemm2m_eisenstein_modulus(int j, int* m, int* s) {
    if (j < 0 || j >= kMaxEis) return GEMM2M_ERR_ARG;
    if (m) *m = eis_modulus_value(j);
    if (s) *s = eis_cube_root(j);
    return GEMM2M_OK;
}

// The rank-k family of Section 5: HERK (B == nullptr) and HER2K on complex inputs; SYRK / SYR2K on real inputs through
// Z = X1 + i X2 (the halves of the k dimension), whose HERK / HER2K has the wanted matrix as its real part.
static int rank_update(int op, int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc,
                       int nmod, void* stream) {
    std::lock_guard<std::mutex> lock(g.mu);
    const bool two = op == GEMM2M_OP_ZHER2K || op == GEMM2M_OP_DSYR2K;
    const bool real_in = op == GEMM2M_OP_DSYRK || op == GEMM2M_OP_DSYR2K;
    if (n < 0 || k < 0) return GEMM2M_ERR_ARG;
    if (lda < (n > 1 ? n : 1) || ldc < (n > 1 ? n : 1) || (two && ldb < (n > 1 ? n : 1))) return GEMM2M_ERR_ARG;
    if (nmod < 1 || nmod > kMax2M) return GEMM2M_ERR_NMOD;    // 2M moduli only: the hybrid serves the complex GEMMs
    if (n > kMaxRows) return GEMM2M_ERR_ARG;
    if (n == 0) return GEMM2M_OK;
    if (!C || (k > 0 && (!A || (two && !B)))) return GEMM2M_ERR_ARG;
    if (int s = check_device()) return s;
    cudaStream_t st = (cudaStream_t)stream;
    Carve c;
    if (!carve(op, n, n, k > 0 ? k : 1, nmod, &c)) return GEMM2M_ERR_ARG;
    if (!D().ws || D().ws_bytes < (size_t)c.total) return GEMM2M_ERR_WORKSPACE;
    char* ws = (char*)D().ws;
    uint64_t* absA = (uint64_t*)(ws + c.off_abs_a);
    int32_t* eA = (int32_t*)(ws + c.off_exp_a);
    int8_t* apm = (int8_t*)(ws + c.off_apm);
    int8_t* bpm = (int8_t*)(ws + c.off_bpm);
    int8_t* cp = (int8_t*)(ws + c.off_cpm);
    const int64_t kc = real_in ? (k + 1) / 2 : k;                   // inner dimension of the complex problem
    // One scale vector for both operands (sigma = tau).  A rank-2k entry is the inner product of two rows of 2 kc complex
    // numbers, so its rows count 2 kc terms in the 2-norm bound.
    const ScaleTargets sc = scale_targets(nmod, two ? 2 * kc : kc, true);
    const bool wide = sc.PA - sc.ck > 62;
    ResidueTable rtab;
    build_residue_table(nmod, &rtab);
    PostMmaTable ptab;
    build_post_mma_table_herk(nmod, &ptab);
    uint32_t* frags = (uint32_t*)(ws + c.off_frags);
    Phases ph;
    if (int s = begin_call(&ph)) return s;
    if (D().frags_key != 128 + nmod) {                       // the operand of the post-processing stays in the workspace between calls
        CK(launch_post_operands(ptab, frags, st, &g.launches[3]));
        D().frags_key = 128 + nmod;
    }
    CK(ph.begin(0, st));
    const double* ZA = A;
    const double* ZB = B;
    int64_t ldza = lda, ldzb = ldb;
    if (real_in && k > 0) {
        CK(launch_pack_real_pair(A, lda, n, k, (double*)(ws + c.off_pack_a), st, &g.launches[0]));
        ZA = (const double*)(ws + c.off_pack_a);
        ldza = n;
        if (two) {
            CK(launch_pack_real_pair(B, ldb, n, k, (double*)(ws + c.off_pack_b), st, &g.launches[0]));
            ZB = (const double*)(ws + c.off_pack_b);
            ldzb = n;
        }
    }
    CK(cudaMemsetAsync(absA, 0, (size_t)8 * n, st));
    CK(launch_scan_rows<double>(ZA, n, k > 0 ? kc : 0, ldza, absA, st, &g.launches[0]));
    if (two) CK(launch_scan_rows<double>(ZB, n, k > 0 ? kc : 0, ldzb, absA, st, &g.launches[0]));
    CK(launch_exponents<double>(absA, n, sc.PA, sc.ck, eA, st, &g.launches[0]));
    CK(ph.end(st));
    CK(ph.begin(1, st));
    if (k == 0) {
        CK(cudaMemsetAsync(apm, 0, (size_t)2 * nmod * n * c.kp, st));
        if (two) CK(cudaMemsetAsync(bpm, 0, (size_t)2 * nmod * n * c.kp, st));
    } else {
        int* dev_status = (int*)(ws + c.off_status);
        if (int s = run_residues<double>(ZA, ldza, false, false, n, kc, c.kp, eA, rtab, wide, apm, dev_status, st)) return s;
        if (two) { if (int s = run_residues<double>(ZB, ldzb, false, false, n, kc, c.kp, eA, rtab, wide, bpm, dev_status, st)) return s; }
    }
    CK(ph.end(st));
    // Section 5.  HERK: C+ = A+ A-^T.  HER2K: C+ = A+ B-^T + B+ A-^T (second product accumulated mod m_j).  C- = C+^T in both.
    // TMEM columns (contiguous index i of the output) <- rows of the "+" planes, TMEM lanes (j) <- rows of the "-" planes,
    // so that out[j][i] = sum_k X+[i,k] Y-[j,k].
    GemmArgs ga;
    ga.R = n; ga.Cn = n; ga.Kp = c.kp;
    ga.row_planes = ga.col_planes = 2 * nmod;
    ga.row_plane0 = nmod;    // "-" planes
    ga.col_plane0 = 0;       // "+" planes
    ga.nbatch = nmod;
    ga.out = cp; ga.ldp = c.ldp;
    build_mod_table(nmod, false, &ga.mods);
    ga.dev_status = (int*)(ws + c.off_status);
    // The output is cut into row panels: entry (i, j) of the lower triangle needs C+[i, j] and C+[j, i], i.e. the GEMM output
    // rows j and i <= the end of i's panel, so the post-processing of the rows of panel p can run on the library's stream
    // beside the GEMMs of panel p + 1 (the last, largest panel stays on the caller's stream).
    if (int s = panel_pipeline(n, st, ph,
            [&](int64_t r0, int64_t r1) {
                ga.row_begin = r0; ga.row_end = r1;
                ga.colop = apm; ga.rowop = two ? bpm : apm; ga.accumulate = 0;
                if (int s = run_gemm(ga, gemm_k_limit(nmod), st)) return s;
                if (two) {
                    ga.colop = bpm; ga.rowop = apm; ga.accumulate = 1;
                    if (int s = run_gemm(ga, gemm_k_limit(nmod), st)) return s;
                }
                return (int)GEMM2M_OK;
            },
            [&](int64_t r0, int64_t r1, cudaStream_t ps) {
                return launch_post_herk(cp, c.ldp, n, r0, r1, eA, ptab, frags, C, ldc, real_in, ps, &g.launches[3]);
            })) return s;
    ph.done();
    return GEMM2M_OK;
}

int zgemm2m_ex(char transa, char transb, int64_t m, int64_t n, int64_t k, const double* alpha, const double* A, int64_t lda,
               const double* B, int64_t ldb, const double* beta, double* C, int64_t ldc, int nmod, void* stream) {
    return xgemm2m<double>(GEMM2M_OP_ZGEMM, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, nmod, stream);
}

int cgemm2m_ex(char transa, char transb, int64_t m, int64_t n, int64_t k, const float* alpha, const float* A, int64_t lda,
               const float* B, int64_t ldb, const float* beta, float* C, int64_t ldc, int nmod, void* stream) {
    double a[2] = {1.0, 0.0}, b[2] = {0.0, 0.0};
    if (alpha) { a[0] = alpha[0]; a[1] = alpha[1]; }
    if (beta) { b[0] = beta[0]; b[1] = beta[1]; }
    return xgemm2m<float>(GEMM2M_OP_CGEMM, transa, transb, m, n, k, a, A, lda, B, ldb, b, C, ldc, nmod, stream);
}

int dgemm_ozaki2(int64_t m, int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc,
                 int nmod, void* stream) {
    std::lock_guard<std::mutex> lock(g.mu);
    if (m < 0 || n < 0 || k < 0) return GEMM2M_ERR_ARG;
    if (lda < (m > 1 ? m : 1) || ldb < (k > 1 ? k : 1) || ldc < (m > 1 ? m : 1)) return GEMM2M_ERR_ARG;
    if (nmod < 1 || nmod > kMaxReal) return GEMM2M_ERR_NMOD;
    if (m > kMaxRows || n > kMaxRows) return GEMM2M_ERR_ARG;
    if (m == 0 || n == 0) return GEMM2M_OK;
    if (!C || (k > 0 && (!A || !B))) return GEMM2M_ERR_ARG;
    if (int s = check_device()) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if (k == 0) {
        CK(cudaMemset2DAsync(C, (size_t)ldc * sizeof(double), 0, (size_t)m * sizeof(double), (size_t)n, st));
        return GEMM2M_OK;
    }
    Carve c;
    if (!carve(GEMM2M_OP_DGEMM_OZAKI2, m, n, k, nmod, &c)) return GEMM2M_ERR_ARG;
    if (!D().ws || D().ws_bytes < (size_t)c.total) return GEMM2M_ERR_WORKSPACE;
    char* ws = (char*)D().ws;
    uint64_t* absA = (uint64_t*)(ws + c.off_abs_a);
    uint64_t* absB = (uint64_t*)(ws + c.off_abs_b);
    int32_t* eA = (int32_t*)(ws + c.off_exp_a);
    int32_t* eB = (int32_t*)(ws + c.off_exp_b);
    int8_t* apl = (int8_t*)(ws + c.off_apm);
    int8_t* bpl = (int8_t*)(ws + c.off_bpm);
    int8_t* cpl = (int8_t*)(ws + c.off_cpm);
    const ScaleTargets sc = scale_targets_real(nmod, k);
    ResidueTable rtab;
    build_residue_table_real(nmod, &rtab);
    CrtTable ctab;
    build_crt_table_real(nmod, &ctab);
    const bool wideA = sc.PA - sc.ck > 62, wideB = sc.PB - sc.ck > 62;
    Phases ph;
    if (int s = begin_call(&ph)) return s;
    // Section 3.1: scale factors, truncation, residues for every modulus, one real int8 GEMM per modulus, CRT, unscale
    CK(ph.begin(0, st));
    CK(cudaMemsetAsync(ws + c.off_abs_a, 0, (size_t)(c.off_exp_a - c.off_abs_a), st));
    CK(launch_scan_real<double>(A, m, k, lda, true, absA, st, &g.launches[0]));
    CK(launch_scan_real<double>(B, k, n, ldb, false, absB, st, &g.launches[0]));
    CK(launch_exponents<double>(absA, m, sc.PA, sc.ck, eA, st, &g.launches[0]));
    CK(launch_exponents<double>(absB, n, sc.PB, sc.ck, eB, st, &g.launches[0]));
    CK(ph.end(st));
    CK(ph.begin(1, st));
    CK(launch_residues_real<double>(A, lda, false, m, k, c.kp, eA, rtab, wideA, apl, st, &g.launches[1]));
    CK(launch_residues_real<double>(B, ldb, true, n, k, c.kp, eB, rtab, wideB, bpl, st, &g.launches[1]));
    CK(ph.end(st));
    GemmArgs ga;
    ga.rowop = bpl; ga.colop = apl;
    ga.R = n; ga.Cn = m; ga.Kp = c.kp;
    ga.row_planes = ga.col_planes = nmod;
    ga.row_plane0 = ga.col_plane0 = 0;
    ga.nbatch = nmod;
    ga.out = cpl; ga.ldp = c.ldp; ga.accumulate = 0;
    build_mod_table_real(nmod, &ga.mods);
    ga.dev_status = (int*)(ws + c.off_status);
    const int64_t klim = gemm_k_limit_real();
    if (int s = panel_pipeline(n, st, ph,
            [&](int64_t j0, int64_t j1) {
                ga.row_begin = j0; ga.row_end = j1;
                return run_gemm(ga, klim, st);
            },
            [&](int64_t j0, int64_t j1, cudaStream_t ps) {
                return launch_post_real(cpl, c.ldp, m, n, j0, j1, eA, eB, ctab, C, ldc, ps, &g.launches[3]);
            })) return s;
    ph.done();
    return GEMM2M_OK;
}

int zherk2m(int64_t n, int64_t k, const double* A, int64_t lda, double* C, int64_t ldc, int nmod, void* stream) {
    return rank_update(GEMM2M_OP_ZHERK, n, k, A, lda, nullptr, 0, C, ldc, nmod, stream);
}

int zher2k2m(int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc, int nmod,
             void* stream) {
    return rank_update(GEMM2M_OP_ZHER2K, n, k, A, lda, B, ldb, C, ldc, nmod, stream);
}

int dsyrk2m(int64_t n, int64_t k, const double* A, int64_t lda, double* C, int64_t ldc, int nmod, void* stream) {
    return rank_update(GEMM2M_OP_DSYRK, n, k, A, lda, nullptr, 0, C, ldc, nmod, stream);
}

int dsyr2k2m(int64_t n, int64_t k, const double* A, int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc, int nmod,
             void* stream) {
    return rank_update(GEMM2M_OP_DSYR2K, n, k, A, lda, B, ldb, C, ldc, nmod, stream);
}

int gemm2m_device_status(void* stream) {
    std::lock_guard<std::mutex> lock(g.mu);
    CK(cudaStreamSynchronize((cudaStream_t)stream));
    select_device();
    if (!D().ws) return GEMM2M_OK;
    int code = 0;
    CK(cudaMemcpy(&code, D().ws, sizeof(int), cudaMemcpyDeviceToHost));
    if (code != kDevOk) {
        CK(cudaMemset(D().ws, 0, sizeof(int)));
        return GEMM2M_ERR_DEVICE_TIMEOUT;
    }
    return GEMM2M_OK;
}

int gemm2m_debug_wait_selftest(uint64_t budget_ns, void* stream) {
    std::lock_guard<std::mutex> lock(g.mu);
    if (int s = check_device()) return s;
    if (!D().ws) return GEMM2M_ERR_WORKSPACE;
    CK(launch_wait_selftest((int*)D().ws, (unsigned long long)budget_ns, (cudaStream_t)stream));
    return GEMM2M_OK;
}

int gemm2m_set_profiling(int enabled) {
    std::lock_guard<std::mutex> lock(g.mu);
    g.profiling = enabled ? 1 : 0;
    g.prof_calls = 0;
    return GEMM2M_OK;
}

int gemm2m_phase_ms(float ms[4], int* calls) {
    std::lock_guard<std::mutex> lock(g.mu);
    const int count = g.prof_calls < State::kProfSlots ? g.prof_calls : State::kProfSlots;
    if (!ms || count == 0) return GEMM2M_ERR_ARG;
    for (int i = 0; i < 4; ++i) ms[i] = 0.f;
    for (int c = 0; c < count; ++c) {
        const State::Slot& slot = g.slots[c];
        for (int i = 0; i < slot.n; ++i) {
            float t = 0.f;
            CK(cudaEventSynchronize(slot.iv[i].b));
            CK(cudaEventElapsedTime(&t, slot.iv[i].a, slot.iv[i].b));
            ms[slot.iv[i].phase] += t / (float)count;
        }
    }
    if (calls) *calls = count;
    return GEMM2M_OK;
}

int gemm2m_last_launch_count(int per_phase[4]) {
    std::lock_guard<std::mutex> lock(g.mu);
    int total = 0;
    for (int i = 0; i < 4; ++i) {
        if (per_phase) per_phase[i] = g.launches[i];
        total += g.launches[i];
    }
    return total;
}

int gemm2m_debug_set_panels(int max_panels) {
    std::lock_guard<std::mutex> lock(g.mu);
    if (max_panels < 1 || max_panels > State::kMaxPanels) return GEMM2M_ERR_ARG;
    g.max_panels = max_panels;
    return GEMM2M_OK;
}

int gemm2m_debug_set_overlap(int enabled) {
    std::lock_guard<std::mutex> lock(g.mu);
    g.overlap = enabled ? 1 : 0;
    return GEMM2M_OK;
}

int gemm2m_debug_set_chained_launch(int enabled) {
    std::lock_guard<std::mutex> lock(g.mu);
    g.chained = enabled ? 1 : 0;
    return GEMM2M_OK;
}

int gemm2m_debug_set_gemm_kernel(int which) {
    std::lock_guard<std::mutex> lock(g.mu);
    if (which < 0 || which > 1) return GEMM2M_ERR_ARG;
    g.gemm_kernel = which;
    return GEMM2M_OK;
}

int gemm2m_set_scaling(int mode) {
    std::lock_guard<std::mutex> lock(g.mu);
    if (mode < 0 || mode > 1) return GEMM2M_ERR_ARG;
    g.scaling = mode;
    return GEMM2M_OK;
}

int gemm2m_debug_tables_real(int nmod, int64_t k, int* moduli, int* scale, double* crt_g, double* crt_m, int* nchunks, int32_t* y0_bits, float* cq,
                             float* inv_m, int32_t* xmax, double* margin) {
    if (nmod < 1 || nmod > kMaxReal || k < 0) return GEMM2M_ERR_ARG;
    const ScaleTargets sc = scale_targets_real(nmod, k);
    if (scale) { scale[0] = sc.Pt; scale[1] = sc.PA; scale[2] = sc.PB; scale[3] = sc.ck; }
    CrtTable ct;
    build_crt_table_real(nmod, &ct);
    ResidueTable rt;
    build_residue_table_real(nmod, &rt);
    for (int j = 0; j < nmod; ++j) {
        if (moduli) moduli[j] = real_modulus_value(j);
        for (int c = 0; c < kMaxChunks; ++c)
            if (crt_g) crt_g[j * kMaxChunks + c] = ct.gr[j][c];
        if (y0_bits) y0_bits[j] = rt.magic[j];
        if (cq) cq[j] = rt.cq[j];
        if (inv_m) inv_m[j] = rt.inv_m[j];
        if (xmax) xmax[j] = rt.xmax[j];
        if (margin) margin[j] = residue_reduction_margin(rt, j);
    }
    if (crt_m) for (int c = 0; c < kMaxChunks; ++c) crt_m[c] = ct.Mc[c];
    if (nchunks) *nchunks = ct.nchunks;
    return GEMM2M_OK;
}

int gemm2m_debug_tables_eisenstein(int nmod, int64_t k, int* scale, double* crt_gr, double* crt_gi, double* crt_m, int* nchunks, int32_t* y0_bits,
                                   float* cq, float* inv_m, int32_t* xmax, double* margin) {
    if (nmod < 1 || nmod > kMaxEis || k < 0) return GEMM2M_ERR_ARG;
    const ScaleTargets sc = scale_targets_eis(nmod, k);
    if (scale) { scale[0] = sc.Pt; scale[1] = sc.PA; scale[2] = sc.PB; scale[3] = sc.ck; }
    CrtTable ct;
    build_crt_table_eis(nmod, &ct);
    ResidueTable rt;
    build_residue_table_eis(nmod, &rt);
    for (int j = 0; j < nmod; ++j) {
        for (int c = 0; c < kMaxChunks; ++c) {
            if (crt_gr) crt_gr[j * kMaxChunks + c] = ct.gr[j][c];
            if (crt_gi) crt_gi[j * kMaxChunks + c] = ct.gi[j][c];
        }
        if (y0_bits) y0_bits[j] = rt.magic[j];
        if (cq) cq[j] = rt.cq[j];
        if (inv_m) inv_m[j] = rt.inv_m[j];
        if (xmax) xmax[j] = rt.xmax[j];
        if (margin) margin[j] = residue_reduction_margin(rt, j);
    }
    if (crt_m) for (int c = 0; c < kMaxChunks; ++c) crt_m[c] = ct.Mc[c];
    if (nchunks) *nchunks = ct.nchunks;
    return GEMM2M_OK;
}

int gemm2m_debug_residue_reduction(int nmod, int32_t* y0_bits, float* cq, float* inv_m, int32_t* xmax, double* margin) {
    if (nmod < 1 || nmod > kMaxMod) return GEMM2M_ERR_ARG;
    ResidueTable rt;
    build_residue_table(nmod, &rt);
    for (int j = 0; j < nmod; ++j) {
        if (y0_bits) y0_bits[j] = rt.magic[j];
        if (cq) cq[j] = rt.cq[j];
        if (inv_m) inv_m[j] = rt.inv_m[j];
        if (xmax) xmax[j] = rt.xmax[j];
        if (margin) margin[j] = residue_reduction_margin(rt, j);
    }
    return GEMM2M_OK;
}

int gemm2m_debug_post_operands(int variant, int nmod, uint8_t* digits, int* dims, double* consts) {
    if (variant < 0 || variant > 2 || nmod < 1 || nmod > (variant == 1 ? kMaxEis : variant == 2 ? kMax2M : kMaxMod)) return GEMM2M_ERR_ARG;
    PostMmaTable t;
    if (variant == 1) build_post_mma_table_eis(nmod, &t);
    else if (variant == 2) build_post_mma_table_herk(nmod, &t);
    else build_post_mma_table(nmod, &t);
    if (dims) { dims[0] = t.c.planes; dims[1] = t.c.ks; dims[2] = t.c.nb; }
    if (digits)
        for (int part = 0; part < 2; ++part)
            for (int p = 0; p < t.c.planes; ++p)
                std::memcpy(digits + ((size_t)part * t.c.planes + p) * 4 * kPostMaxNB, t.digit[part][p], 4 * kPostMaxNB);
    if (consts) {
        for (int k = 0; k < kPostMaxNB; ++k) {
            consts[k] = t.c.Mc[k];
            consts[kPostMaxNB + k] = t.c.off[0][k];
            consts[2 * kPostMaxNB + k] = t.c.off[1][k];
        }
        consts[3 * kPostMaxNB] = t.c.inv_M;
    }
    return GEMM2M_OK;
}

int gemm2m_debug_tables(int nmod, int64_t k, int herk, int* scale, double* crt_gr, double* crt_gi, double* crt_m, int* nchunks,
                        int8_t* res_w) {
    if (nmod < 1 || nmod > kMaxMod || k < 0) return GEMM2M_ERR_ARG;
    const ScaleTargets sc = scale_targets(nmod, k, herk != 0);
    if (scale) { scale[0] = sc.Pt; scale[1] = sc.PA; scale[2] = sc.PB; scale[3] = sc.ck; }
    CrtTable ct;
    build_crt_table(nmod, &ct);
    for (int j = 0; j < nmod; ++j)
        for (int c = 0; c < kMaxChunks; ++c) {
            if (crt_gr) crt_gr[j * kMaxChunks + c] = ct.gr[j][c];
            if (crt_gi) crt_gi[j * kMaxChunks + c] = ct.gi[j][c];
        }
    if (crt_m) for (int c = 0; c < kMaxChunks; ++c) crt_m[c] = ct.Mc[c];
    if (nchunks) *nchunks = ct.nchunks;
    if (res_w) {
        ResidueTable rt;
        build_residue_table(nmod, &rt);
        for (int j = 0; j < nmod; ++j)
            for (int b = 0; b < 8; ++b) {
                const uint32_t w = b < 4 ? rt.w_lo[j] >> (8 * b) : rt.w_hi[j] >> (8 * (b - 4));
                const uint32_t ws = b < 4 ? rt.ws_lo[j] >> (8 * b) : rt.ws_hi[j] >> (8 * (b - 4));
                res_w[j * 16 + b] = (int8_t)(w & 0xFF);
                res_w[j * 16 + 8 + b] = (int8_t)(ws & 0xFF);
            }
    }
    return GEMM2M_OK;
}

}  // extern "C"

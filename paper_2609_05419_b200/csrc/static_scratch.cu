// gemm2m_zscale_exponents_static: the scale-exponent computation of zgemm2m (Algorithm 1 step 2) for callers that
// cannot allocate device memory.  Its scratch (one 64-bit maximum per row of A) lives in a file-scope device array
// instead of a caller-provided workspace, so the call needs nothing but its input and output.
#include "../../include/gemm2m.h"

#include "common.cuh"

#include <mutex>

using namespace gemm2m;

namespace {

// Scratch for the per-row maxima.  Every GPU that loads this library holds these 512 KB until the process exits.
// All calls share it and it keeps the last call's contents: the entry point clears the part it uses before the scan.
static __device__ __align__(256) unsigned long long g_static_absmax[GEMM2M_STATIC_MAX_ROWS];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned long long* g_scratch_addr[kMaxDevices] = {};   // device address of g_static_absmax, per device
int g_arch_ok[kMaxDevices] = {};                        // 0 = not asked yet, 1 = compute capability 10.0, -1 = anything else

// In host code the name g_static_absmax is only a handle, not a device address: handing it to a kernel would make
// the kernel read and write some unrelated location.  The address on the current device comes from the runtime.
cudaError_t scratch_for_current_device(unsigned long long** out, bool* arch_ok) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_arch_ok[dev]) {
        int major = 0, minor = 0;
        err = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (err == cudaSuccess) err = cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev);
        if (err != cudaSuccess) return err;
        g_arch_ok[dev] = (major == 10 && minor == 0) ? 1 : -1;
    }
    *arch_ok = g_arch_ok[dev] > 0;
    if (!*arch_ok) return cudaSuccess;                     // the kernels exist for this architecture only
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        err = cudaGetSymbolAddress(&p, g_static_absmax);   // set-up, once per device, with that device current
        if (err != cudaSuccess) return err;
        g_scratch_addr[dev] = static_cast<unsigned long long*>(p);
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int gemm2m_zscale_exponents_static(int64_t m, int64_t k, const double* A, int64_t lda, int nmod, int32_t* e, void* stream) {
    if (m < 0 || k < 0 || lda < (m > 1 ? m : 1)) return GEMM2M_ERR_ARG;
    if (nmod < 1 || nmod > kMaxMod) return GEMM2M_ERR_NMOD;
    if (m > GEMM2M_STATIC_MAX_ROWS) return GEMM2M_ERR_WORKSPACE;   // the built-in scratch is too small for this many rows
    if (m == 0) return GEMM2M_OK;
    if (!e || (k > 0 && !A)) return GEMM2M_ERR_ARG;
    unsigned long long* scratch = nullptr;
    bool arch_ok = false;
    if (scratch_for_current_device(&scratch, &arch_ok) != cudaSuccess) return GEMM2M_ERR_CUDA;
    if (!arch_ok) return GEMM2M_ERR_ARCH;
    cudaStream_t st = (cudaStream_t)stream;
    const ScaleTargets sc = scale_targets(nmod, k, false);
    int launches = 0;
    // the maxima are accumulated with atomicMax, so they must start at zero on every call
    if (cudaMemsetAsync(scratch, 0, sizeof(unsigned long long) * (size_t)m, st) != cudaSuccess) return GEMM2M_ERR_CUDA;
    if (launch_scan_rows<double>(A, m, k, lda, reinterpret_cast<uint64_t*>(scratch), st, &launches) != cudaSuccess) return GEMM2M_ERR_CUDA;
    if (launch_exponents<double>(reinterpret_cast<const uint64_t*>(scratch), m, sc.PA, sc.ck, e, st, &launches) != cudaSuccess)
        return GEMM2M_ERR_CUDA;
    return GEMM2M_OK;
}

// Device and host helpers shared by the scan, residue and post-processing kernels.
#pragma once
#include "common.cuh"

namespace gemm2m {

template <typename T> struct FpBits;
template <> struct FpBits<double> {
    using U = unsigned long long;
    static constexpr int kMantBits = 52, kExpMax = 2047, kBias = 1023;
    __device__ static U mag(double v) { return (U)__double_as_longlong(v) & 0x7FFFFFFFFFFFFFFFull; }
};
template <> struct FpBits<float> {
    using U = unsigned long long;
    static constexpr int kMantBits = 23, kExpMax = 255, kBias = 127;
    __device__ static U mag(float v) { return (U)(__float_as_uint(v) & 0x7FFFFFFFu); }
};

// Scale exponent of a row / column from the bit pattern of its largest |Re| or |Im| (Algorithm 1 step 2):
// e = floor(log2 mu) + 1 + c_k - P; 0 for an all-zero row; the sentinel for a row that holds an Inf or NaN.
template <typename T>
__device__ __forceinline__ int scale_exponent(unsigned long long absmax_bits, int P, int ck) {
    if (absmax_bits == 0) return 0;
    const int E = (int)(absmax_bits >> FpBits<T>::kMantBits);
    if (E == FpBits<T>::kExpMax) return kExpNonFinite;
    const int x = E ? E - FpBits<T>::kBias : (63 - __clzll((long long)absmax_bits)) - (FpBits<T>::kBias - 1 + FpBits<T>::kMantBits);
    return x + 1 + ck - P;
}

template <typename T> struct Cplx { T re, im; };
template <typename T> __device__ __forceinline__ Cplx<T> load_cplx(const T* p);
template <> __device__ __forceinline__ Cplx<double> load_cplx<double>(const double* p) {
    const double2 v = __ldg(reinterpret_cast<const double2*>(p));
    return {v.x, v.y};
}
template <> __device__ __forceinline__ Cplx<float> load_cplx<float>(const float* p) {
    const float2 v = __ldg(reinterpret_cast<const float2*>(p));
    return {v.x, v.y};
}

inline int cached_sm_count() {
    static int sms_dev[kMaxDevices] = {};
    int& sms = sms_dev[current_device_slot()];
    if (!sms) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            sms = 148;
    }
    return sms;
}

}  // namespace gemm2m

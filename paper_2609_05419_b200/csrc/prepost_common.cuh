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

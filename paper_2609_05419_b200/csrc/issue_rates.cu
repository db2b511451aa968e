// Measures how many lanes per SM and cycle this GPU sustains for the instruction kinds the pre- and post-processing kernels
// are made of: streams of independent instructions (8 chains per thread, 32 warps per SM), timed with CUDA events.  A
// stand-alone program (not part of the library): it backs the dispatch-cycle accounts of those kernels.
#include <cstdint>
#include <cstdio>
#include <cuda_runtime.h>

enum Kind { FFMA, FADD, LEA, IADD, IMAD, IDP4A, PRMT, SHF, IMADWIDE, IMADHI, DFMA, DADD, DMUL, kKinds };
static const char* kNames[kKinds] = {"FFMA", "FADD", "LEA (shift + add)", "IADD", "IMAD", "IDP.4A", "PRMT", "SHF", "IMAD.WIDE", "IMAD.HI",
                                     "DFMA", "DADD", "DMUL"};

template <int KIND>
__global__ void stream_kernel(uint32_t* out, int iters, uint32_t a, uint32_t b, double da, double db) {
    uint32_t x[8];
    double d[8];
    for (int i = 0; i < 8; ++i) { x[i] = threadIdx.x * 2654435761u + i; d[i] = threadIdx.x * 1e-3 + i; }
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (KIND == FFMA) x[i] = __float_as_uint(fmaf(__uint_as_float(x[i]), __uint_as_float(a), __uint_as_float(b)));
            else if (KIND == FADD) x[i] = __float_as_uint(__uint_as_float(x[i]) + __uint_as_float(a));
            else if (KIND == LEA) x[i] = (x[i] << 3) + a;
            else if (KIND == IADD) x[i] = x[i] + (a ^ (uint32_t)it);
            else if (KIND == IMAD) x[i] = x[i] * a + b;
            else if (KIND == IDP4A) x[i] = (uint32_t)__dp4a((int)x[i], (int)a, (int)x[i]);
            else if (KIND == PRMT) x[i] = __byte_perm(x[i], a, 0x5140 ^ (b & 0x7777));
            else if (KIND == SHF) x[i] = __funnelshift_l(x[i], a, 7);
            else if (KIND == IMADWIDE) { const unsigned long long w = (unsigned long long)x[i] * a + b; x[i] = (uint32_t)w ^ (uint32_t)(w >> 32); }
            else if (KIND == IMADHI) x[i] = __umulhi(x[i], a);
            else if (KIND == DFMA) d[i] = fma(d[i], da, db);
            else if (KIND == DADD) d[i] = d[i] + da;
            else if (KIND == DMUL) d[i] = d[i] * da;
        }
    }
    uint32_t s = 0;
    for (int i = 0; i < 8; ++i) s += x[i] + (uint32_t)__double2loint(d[i]);
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

template <int KIND>
static void run(uint32_t* out, int sms, double ghz) {
    const int threads = 256, blocks = sms * 4, iters = 20000;
    stream_kernel<KIND><<<blocks, threads>>>(out, 100, 0x01020304u, 7u, 1.0000001, 1e-9);
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    cudaEventRecord(e0);
    stream_kernel<KIND><<<blocks, threads>>>(out, iters, 0x01020304u, 7u, 1.0000001, 1e-9);
    cudaEventRecord(e1);
    cudaEventSynchronize(e1);
    float ms = 0;
    cudaEventElapsedTime(&ms, e0, e1);
    const double lanes_per_ns = (double)blocks * threads * iters * 8 / ms / 1e6 / sms;
    // IMAD.WIDE carries one logic instruction per multiply-add in this loop; the figure is for the pair
    printf("%-18s %8.3f ms  %7.1f lanes per SM and ns  = %6.1f per SM and cycle at %.2f GHz\n", kNames[KIND], ms, lanes_per_ns, lanes_per_ns / ghz, ghz);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
}

int main() {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, 0) != cudaSuccess) { printf("no CUDA device\n"); return 1; }
    const int sms = prop.multiProcessorCount;
    int khz = 0;
    cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, 0);
    const double ghz = khz / 1e6;
    uint32_t* out = nullptr;
    cudaMalloc(&out, sizeof(uint32_t) * 256 * sms * 4);
    printf("%s, %d SMs, nominal SM clock %.3f GHz (the clock during the run may be lower)\n", prop.name, sms, ghz);
    run<FFMA>(out, sms, ghz); run<FADD>(out, sms, ghz); run<LEA>(out, sms, ghz); run<IADD>(out, sms, ghz); run<IMAD>(out, sms, ghz);
    run<IDP4A>(out, sms, ghz); run<PRMT>(out, sms, ghz); run<SHF>(out, sms, ghz); run<IMADWIDE>(out, sms, ghz); run<IMADHI>(out, sms, ghz);
    run<DFMA>(out, sms, ghz); run<DADD>(out, sms, ghz); run<DMUL>(out, sms, ghz);
    const cudaError_t err = cudaDeviceSynchronize();
    cudaFree(out);
    if (err != cudaSuccess) { printf("CUDA error: %s\n", cudaGetErrorString(err)); return 1; }
    return 0;
}

// Measurement aid (see umlmd_probe_fma_peak in umlmd.h): a register-resident chain of
// fused multiply-adds on every FP32 lane of the device, timed with CUDA events, to give the
// edge kernels' roofline a measured denominator instead of one derived from unit counts.
#include <cuda_runtime.h>

#include "../../include/umlmd.h"

namespace {

constexpr int kChains = 8;        // independent accumulators per thread (covers the FMA latency)
constexpr int kIters = 4096;

__global__ void __launch_bounds__(256) k_ffma_probe(float* out, float a, float b) {
    float x[kChains];
#pragma unroll
    for (int k = 0; k < kChains; ++k) x[k] = (float)(threadIdx.x + k) * 1e-3f;
#pragma unroll 1
    for (int i = 0; i < kIters; i += 4) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int k = 0; k < kChains; ++k) x[k] = fmaf(x[k], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < kChains; ++k) s += x[k];
    if (s == 12345.678f) out[0] = s;      // never true for the arguments used; keeps the chain alive
}

}  // namespace

extern "C" int umlmd_probe_fma_peak(double* tflops, void* stream) {
    if (!tflops) return UMLMD_E_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return UMLMD_E_CUDA;
    float* d_out = nullptr;
    if (cudaMalloc(&d_out, sizeof(float)) != cudaSuccess) return UMLMD_E_CUDA;
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    const int blocks = sms * 32, threads = 256;
    double best = 0.0;
    for (int rep = 0; rep < 5; ++rep) {     // first repetition warms up; the best of the rest counts
        cudaEventRecord(e0, st);
        k_ffma_probe<<<blocks, threads, 0, st>>>(d_out, 0.999f, 1e-3f);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess) { best = -1.0; break; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double flops = 2.0 * kChains * kIters * (double)threads * blocks;
        if (rep > 0 && ms > 0.f && flops / (ms * 1e-3) / 1e12 > best) best = flops / (ms * 1e-3) / 1e12;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(d_out);
    if (best <= 0.0) return UMLMD_E_CUDA;
    *tflops = best;
    return UMLMD_OK;
}

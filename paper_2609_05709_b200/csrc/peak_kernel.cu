// Measurement aid: the FP32 multiply-add rate this GPU sustains from registers alone, the denominator of the
// roofline of the descriptor-only build (which is bound by FP32 arithmetic, not by memory).
#include <cuda_runtime.h>

#include "soap.h"

namespace {

constexpr int kChains = 16;       // independent accumulators per thread (covers the 4-cycle FMA latency many times over)
constexpr int kInner = 64;        // multiply-adds per chain and loop trip

__global__ void __launch_bounds__(256) fma_loop_kernel(int trips, float seed, float* sink) {
    float acc[kChains];
#pragma unroll
    for (int k = 0; k < kChains; ++k) acc[k] = seed + (float)(threadIdx.x + k);
    const float a = 1.0f - seed, b = seed;
    for (int t = 0; t < trips; ++t) {
#pragma unroll
        for (int i = 0; i < kInner; ++i)
#pragma unroll
            for (int k = 0; k < kChains; ++k) acc[k] = fmaf(acc[k], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < kChains; ++k) s += acc[k];
    if (s == 12345.678f) sink[blockIdx.x * blockDim.x + threadIdx.x] = s;      // never true: keeps the loop alive
}

}  // namespace

extern "C" int soap_measure_fp32_peak(double* tflops, double* milliseconds, void* stream) {
    if (!tflops) return SOAP_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SOAP_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SOAP_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return SOAP_ERR_CUDA;
    const int blocks = sms * 8, trips = 2048;
    float best = 0.f;
    for (int rep = 0; rep < 5; ++rep) {            // the first repetitions warm the clocks up; the best one counts
        cudaEventRecord(e0, st);
        fma_loop_kernel<<<blocks, 256, 0, st>>>(trips, 0.25f, nullptr);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess) { cudaEventDestroy(e0); cudaEventDestroy(e1); return SOAP_ERR_CUDA; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (rep > 0 && (best == 0.f || ms < best)) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (cudaGetLastError() != cudaSuccess || !(best > 0.f)) return SOAP_ERR_CUDA;
    const double flops = 2.0 * (double)blocks * 256.0 * kChains * kInner * (double)trips;
    *tflops = flops / ((double)best * 1e-3) / 1e12;
    if (milliseconds) *milliseconds = best;
    return SOAP_OK;
}

// FP32 FMA peak probe: the roofline of this library is stated against the plain FP32 FMA rate, so the benchmark
// measures that rate on the device it runs on instead of trusting the nominal clock.
#include "../../include/sna.h"

#include <cuda_runtime.h>

namespace {

constexpr int ITERS = 4096, CHAINS = 16, THREADS = 1024;

__global__ void __launch_bounds__(THREADS) fma_probe_kernel(float* sink, float a, float b) {
    float acc[CHAINS];
#pragma unroll
    for (int i = 0; i < CHAINS; ++i) acc[i] = threadIdx.x * 1e-3f + i;
    for (int it = 0; it < ITERS; ++it) {
#pragma unroll
        for (int i = 0; i < CHAINS; ++i) acc[i] = fmaf(acc[i], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < CHAINS; ++i) s += acc[i];
    if (s == 12345.678f) sink[0] = s;   // keeps the loop alive; practically never true
}

}  // namespace

extern "C" sna_status_t sna_measure_fp32_fma_peak(double* tflops) {
    if (tflops == nullptr) return SNA_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SNA_ERR_CUDA;
    float* sink = nullptr;
    if (cudaMalloc(&sink, 256) != cudaSuccess) return SNA_ERR_ALLOC;
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    const int blocks = sms * 2;   // two full CTAs per SM keep every scheduler supplied with independent FMAs
    float best_ms = 1e30f;
    for (int rep = 0; rep < 5; ++rep) {
        cudaEventRecord(e0);
        fma_probe_kernel<<<blocks, THREADS>>>(sink, 1.0001f, 0.5f);
        cudaEventRecord(e1);
        if (cudaEventSynchronize(e1) != cudaSuccess) { cudaFree(sink); return SNA_ERR_CUDA; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (rep > 0 && ms < best_ms) best_ms = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(sink);
    if (cudaGetLastError() != cudaSuccess) return SNA_ERR_CUDA;
    const double flops = 2.0 * (double)blocks * THREADS * ITERS * CHAINS;
    *tflops = flops / (best_ms * 1e-3) / 1e12;
    return SNA_OK;
}

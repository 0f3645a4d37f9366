// Measurement utility: fp32 FMA rate of the device, for the roofline denominator
// of kernels bound by plain ALU arithmetic.
#include "common.cuh"

namespace {

constexpr int PEAK_ITERS = 4096;
constexpr int CHAINS = 16;

__global__ void __launch_bounds__(256) fma_loop_kernel(float *sink, float a, float b) {
    float x[CHAINS];
#pragma unroll
    for (int i = 0; i < CHAINS; ++i) x[i] = (float)(threadIdx.x + i) * 1e-3f;
    for (int it = 0; it < PEAK_ITERS; ++it) {
#pragma unroll
        for (int i = 0; i < CHAINS; ++i) x[i] = fmaf(x[i], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < CHAINS; ++i) s += x[i];
    if (s == 123.456f) sink[0] = s;   // never true in practice; keeps the loop alive
}

}  // namespace

extern "C" int aug_measure_fp32_peak(void *cuda_stream, float *tflops_host) {
    if (!tflops_host) return AUG_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int dev = 0, sms = 0;
    AUG_CUDA_OK(cudaGetDevice(&dev));
    AUG_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    float *sink = nullptr;
    AUG_CUDA_OK(cudaMalloc(&sink, sizeof(float)));
    cudaEvent_t e0, e1;
    AUG_CUDA_OK(cudaEventCreate(&e0));
    AUG_CUDA_OK(cudaEventCreate(&e1));
    const int blocks = sms * 32;
    float best = 0.f;
    for (int rep = 0; rep < 4; ++rep) {   // first repetition warms up
        cudaEventRecord(e0, st);
        fma_loop_kernel<<<blocks, 256, 0, st>>>(sink, 0.999f, 1e-4f);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess) break;
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double flop = 2.0 * CHAINS * (double)PEAK_ITERS * 256.0 * blocks;
        const float tf = (float)(flop / (ms * 1e-3) / 1e12);
        if (rep > 0 && tf > best) best = tf;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(sink);
    AUG_CUDA_OK(cudaGetLastError());
    *tflops_host = best;
    return AUG_OK;
}

// Measured fp32 FMA rate of the device: the denominator of the fused kernel's roofline, taken in the
// same process and at the same clocks as the kernel it is compared with.  Every thread runs eight
// independent FMA chains; the grid fills every SM with the maximum number of resident warps.
#include "common.cuh"

namespace mlip {

constexpr int PEAK_CHAINS = 8;
constexpr int PEAK_ITERS = 4096;

__global__ void __launch_bounds__(1024) k_ffma_peak(float *out, float a, float b) {
    float x[PEAK_CHAINS];
#pragma unroll
    for (int c = 0; c < PEAK_CHAINS; ++c) x[c] = (float)(threadIdx.x + c);
    for (int it = 0; it < PEAK_ITERS; ++it) {
#pragma unroll
        for (int c = 0; c < PEAK_CHAINS; ++c) x[c] = fmaf(x[c], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < PEAK_CHAINS; ++c) s += x[c];
    if (s == 123.456f) out[0] = s;   // never true for the arguments used; keeps the chains alive
}

}  // namespace mlip

extern "C" int mlip_measure_fp32_peak(int device, double *tflops_host) {
    using namespace mlip;
    if (!tflops_host) return MLIP_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    if (cudaSetDevice(device) != cudaSuccess || cudaGetDeviceProperties(&prop, device) != cudaSuccess) return MLIP_ERR_CUDA;
    float *out = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int rc = MLIP_ERR_CUDA;
    do {
        if (cudaMalloc(&out, sizeof(float)) != cudaSuccess) break;
        if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) break;
        const int blocks = prop.multiProcessorCount * 2 * 8;   // 2 resident CTAs of 1024 threads per SM, 8 waves
        double best = 0.0;
        for (int rep = 0; rep < 5; ++rep) {   // first repetition warms up
            cudaEventRecord(e0, 0);
            k_ffma_peak<<<blocks, 1024>>>(out, 0.999f, 0.001f);
            cudaEventRecord(e1, 0);
            if (cudaEventSynchronize(e1) != cudaSuccess) break;
            float ms = 0.f;
            cudaEventElapsedTime(&ms, e0, e1);
            const double flop = 2.0 * PEAK_CHAINS * PEAK_ITERS * 1024.0 * blocks;
            if (rep > 0 && ms > 0.f && flop / (ms * 1e-3) / 1e12 > best) best = flop / (ms * 1e-3) / 1e12;
        }
        if (cudaGetLastError() != cudaSuccess || best == 0.0) break;
        *tflops_host = best;
        rc = MLIP_OK;
    } while (0);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(out);
    return rc;
}

// Two micro-benchmarks behind gmm_probe_rates: the rates the secondary roofs of the EM iteration are quoted against.
//   fp32 FMA   every thread runs 8 independent chains of dependent fused multiply-adds (enough to fill the pipeline at
//              the occupancy used); the figure is 2 flop per FMA.  This is the roof of the FP32 (CUDA-core) path.
//   ex2        every thread runs 8 independent chains of ex2.approx.ftz.f32 (the instruction the softmax uses): the
//              special-function unit's rate, the roof of the N K exponentials per iteration.
// Both are timed with CUDA events over a launch of several milliseconds, after a warm-up launch.
#include "internal.cuh"

namespace {

constexpr int PR_THREADS = 256, PR_ITERS = 4096;

__global__ void __launch_bounds__(PR_THREADS) fma_rate_kernel(float* out, float a, float b) {
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = (float)(threadIdx.x + j) * 1e-3f;
    for (int i = 0; i < PR_ITERS; ++i) {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = fmaf(v[j], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) s += v[j];
    if (s == 12345.678f) out[0] = s;          // keeps the chains alive, practically never true
}

__global__ void __launch_bounds__(PR_THREADS) ex2_rate_kernel(float* out, float c) {
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = -(float)(threadIdx.x + j) * 1e-3f;
    for (int i = 0; i < PR_ITERS; ++i) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float y;
            asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(v[j]));
            v[j] = y - c;                     // stays in (-1, 0]: one FADD per ex2, on another pipe
        }
    }
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) s += v[j];
    if (s == 12345.678f) out[0] = s;
}

}  // namespace

extern "C" int gmm_probe_rates(int device, double* fp32_fma_flops, double* ex2_per_s) {
    if (!fp32_fma_flops || !ex2_per_s) return GMM_EINVAL;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return GMM_ECUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return GMM_ECUDA; }
    int rc = GMM_OK, sms = 0;
    float* out = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || cudaMalloc(&out, 256) != cudaSuccess ||
        cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        rc = GMM_ECUDA;
    } else {
        const int blocks = sms * 8;           // 8 x 256 threads per SM: full occupancy
        const double per_launch = (double)blocks * PR_THREADS * PR_ITERS * 8.0;
        float ms = 0.f;
        for (int rep = 0; rep < 2; ++rep) {   // the first launch of each is the warm-up
            cudaEventRecord(e0);
            for (int r = 0; r < 4; ++r) fma_rate_kernel<<<blocks, PR_THREADS>>>(out, 0.999f, 1e-3f);
            cudaEventRecord(e1);
            if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) rc = GMM_ECUDA;
        }
        *fp32_fma_flops = ms > 0.f ? 2.0 * 4.0 * per_launch / (ms * 1e-3) : 0.0;
        for (int rep = 0; rep < 2; ++rep) {
            cudaEventRecord(e0);
            for (int r = 0; r < 4; ++r) ex2_rate_kernel<<<blocks, PR_THREADS>>>(out, 1.0f);
            cudaEventRecord(e1);
            if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) rc = GMM_ECUDA;
        }
        *ex2_per_s = ms > 0.f ? 4.0 * per_launch / (ms * 1e-3) : 0.0;
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (out) cudaFree(out);
    if (cudaGetLastError() != cudaSuccess) rc = GMM_ECUDA;
    if (prev != device) cudaSetDevice(prev);
    return rc;
}

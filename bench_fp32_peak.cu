// Register-only FP32 multiply-add throughput probe for bench.py: the measured denominator of the
// "alu" roofline.  Not part of the ConvAttn library; built into its own small shared object.
//
// Every thread runs kChains independent dependency chains of fused multiply-adds for `iters` rounds,
// once with scalar fma.rn.f32 and once with the packed fma.rn.f32x2 of sm_100; nothing touches memory
// until the final (never taken in practice) store that keeps the compiler from dropping the chains.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr int kChains = 16;
constexpr int kThreads = 512;

__global__ void __launch_bounds__(kThreads) fma_scalar(int iters, float seed, float* sink) {
    float a[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) a[c] = seed + (float)(threadIdx.x + c);
    const float m = 0.999f, b = 0.001f;
#pragma unroll 1
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int r = 0; r < 8; ++r)
#pragma unroll
            for (int c = 0; c < kChains; ++c) a[c] = fmaf(a[c], m, b);
    }
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < kChains; ++c) s += a[c];
    if (s == 12345.678f) sink[blockIdx.x * kThreads + threadIdx.x] = s;
}

__global__ void __launch_bounds__(kThreads) fma_packed(int iters, float seed, float* sink) {
    unsigned long long a[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) {
        const float lo = seed + (float)(threadIdx.x + c), hi = lo + 0.5f;
        asm("mov.b64 %0, {%1, %2};" : "=l"(a[c]) : "f"(lo), "f"(hi));
    }
    unsigned long long m, b;
    asm("mov.b64 %0, {%1, %1};" : "=l"(m) : "f"(0.999f));
    asm("mov.b64 %0, {%1, %1};" : "=l"(b) : "f"(0.001f));
#pragma unroll 1
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < kChains; ++c) asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(a[c]) : "l"(m), "l"(b));
    }
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < kChains; ++c) {
        float lo, hi;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a[c]));
        s += lo + hi;
    }
    if (s == 12345.678f) sink[blockIdx.x * kThreads + threadIdx.x] = s;
}

}  // namespace

// Runs both probes on the current device and stream 0.  out[0], out[1]: TFLOP/s (2 flop per multiply-add)
// of the scalar and of the packed form, best of `reps` launches of about `iters` x 128 multiply-adds per
// thread; out[2]: SM count; out[3]: blocks resident per SM that the launch used.  Returns 0, or the CUDA
// error code.  `sink` is a device buffer the function allocates and frees itself.
extern "C" int fp32_peak_measure(int iters, int reps, double* out) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return (int)e;
    const int per_sm = 2;                                    // 2 x 512 threads: 8 warps per scheduler
    const int blocks = sms * per_sm;
    float* sink = nullptr;
    e = cudaMalloc(&sink, (size_t)blocks * kThreads * sizeof(float));
    if (e != cudaSuccess) return (int)e;
    cudaEvent_t a, b;
    cudaEventCreate(&a);
    cudaEventCreate(&b);
    double best[2] = {0.0, 0.0};
    for (int which = 0; which < 2; ++which) {
        for (int r = 0; r < reps + 1; ++r) {                 // first launch is the warm-up
            cudaEventRecord(a, 0);
            if (which == 0) fma_scalar<<<blocks, kThreads>>>(iters, 1.0f, sink);
            else fma_packed<<<blocks, kThreads>>>(iters, 1.0f, sink);
            cudaEventRecord(b, 0);
            e = cudaEventSynchronize(b);
            if (e != cudaSuccess) break;
            float ms = 0.f;
            cudaEventElapsedTime(&ms, a, b);
            const double fmas = (double)blocks * kThreads * (double)iters * 8.0 * kChains;   // both forms: 128 per round
            const double tf = 2.0 * fmas / (ms * 1e-3) / 1e12;
            if (r > 0 && tf > best[which]) best[which] = tf;
        }
        if (e != cudaSuccess) break;
    }
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    cudaFree(sink);
    if (e != cudaSuccess) return (int)e;
    out[0] = best[0];
    out[1] = best[1];
    out[2] = (double)sms;
    out[3] = (double)per_sm;
    return 0;
}

// Backward pass of the module's closing 1x1 convolution (ESC paper, Eq. 4 line 4, with the block's residual, Eq. 3
// line 3):  out = W_fuse cat + b_fuse + residual  per pixel.  With go = dL/dout:
//
//   g_cat[c]  = sum_n W_fuse[n,c] go[n]          per pixel: the forward's 1x1 kernels with the transposed matrix
//   g_W[n,c]  = sum_pixels go[n] cat[c]          kernel wgrad
//   g_b[n]    = sum_pixels go[n]                 kernel wgrad
//   (the residual's gradient is go itself)
//
// wgrad: a block takes a run of pixels, 256 per pass; both tensors' channels are staged channel-major as fp32; the C x C
// pairs are cut into 4x4 register tiles whose rows are C/4 apart (lanes then read adjacent rows: no bank conflicts),
// the pass's pixels into interleaved slices where there are fewer tiles than threads; eight 16-byte reads per 64 FMAs.
// Blocks write their sums once; `sum_wgrad` adds them in block order.
#pragma once
#include "common.cuh"

namespace esc { namespace fuse { namespace bwd {

constexpr int kThreads = 256;
constexpr int kPitch = kThreads + 4;          // floats per staged channel row

template <int C> struct Geom {
    static constexpr int Q = C / 4;                               // rows of a tile are Q apart
    static constexpr int kTiles = Q * Q;
    static constexpr int kSlices = kTiles >= kThreads ? 1 : kThreads / kTiles;
    static constexpr int kPx = kThreads / kSlices;                // pixels per slice and pass
    static constexpr int kPart = C * C + C;                       // floats a block writes: g_W, then g_b
    static constexpr size_t kSmemBytes = (size_t)2 * C * kPitch * sizeof(float);
    static_assert(C % 4 == 0 && kTiles <= kThreads && kPx % 4 == 0 && kSlices * C * C <= 2 * C * kPitch, "tiling");
};

inline bool supported(int C) { return C == 16 || C == 32 || C == 48 || C == 64; }

template <typename T>
__global__ void __launch_bounds__(256)
transpose_w(const T* __restrict__ w, int C, T* __restrict__ wt)
{
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e < C * C) wt[(size_t)(e % C) * C + e / C] = w[e];
}

template <typename T, int LAYOUT, int C>
__global__ void __launch_bounds__(kThreads)
wgrad(const T* __restrict__ cat, const T* __restrict__ go, long long HW, long long pixels, int passes,
      float* __restrict__ part)                                   // [gridDim.x][C * C + C]
{
    using G = Geom<C>;
    extern __shared__ __align__(16) float sm[];
    float* gs = sm;                                               // go  [C][kPitch]
    float* xs = sm + C * kPitch;                                  // cat [C][kPitch]
    const int tid = threadIdx.x;
    const int tile = tid / G::kSlices, slice = tid % G::kSlices;
    const bool active = tile < G::kTiles;
    const int nn = tile / G::Q, kk = tile % G::Q;
    auto index = [&](long long px, int c) -> size_t {
        const long long b = px / HW, r = px - b * HW;
        return LAYOUT == kNCHW ? ((size_t)b * C + c) * HW + r : (size_t)px * C + c;
    };
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    float gb = 0.f;
    for (int pass = 0; pass < passes; ++pass) {
        const long long px0 = ((long long)blockIdx.x * passes + pass) * kThreads;
        if (px0 >= pixels) break;
        __syncthreads();                                          // the last pass's rows are read
        for (int e = tid; e < C * kThreads; e += kThreads) {
            const int r = LAYOUT == kNCHW ? e % kThreads : e / C, c = LAYOUT == kNCHW ? e / kThreads : e % C;
            const long long px = px0 + r;
            float a = 0.f, b = 0.f;
            if (px < pixels) {
                const size_t idx = index(px, c);
                a = Elem<T>::to_f32(go[idx]);
                b = Elem<T>::to_f32(cat[idx]);
            }
            gs[c * kPitch + r] = a;
            xs[c * kPitch + r] = b;
        }
        __syncthreads();
        if (tid < C) {
            const float4* row = reinterpret_cast<const float4*>(gs + tid * kPitch);
            float s = gb;
#pragma unroll 4
            for (int i = 0; i < kThreads / 4; ++i) { const float4 v = row[i]; s += v.x; s += v.y; s += v.z; s += v.w; }
            gb = s;
        }
        if (active) {
#pragma unroll 2
            for (int i = 0; i < G::kPx / 4; ++i) {
                const int px = slice * 4 + i * 4 * G::kSlices;
                float4 u[4], w[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    u[r] = *reinterpret_cast<const float4*>(gs + (nn + r * G::Q) * kPitch + px);
                    w[r] = *reinterpret_cast<const float4*>(xs + (kk + r * G::Q) * kPitch + px);
                }
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float t = acc[r][c];
                        t = fmaf(u[r].x, w[c].x, t); t = fmaf(u[r].y, w[c].y, t);
                        t = fmaf(u[r].z, w[c].z, t); t = fmaf(u[r].w, w[c].w, t);
                        acc[r][c] = t;
                    }
            }
        }
    }
    float* out = part + (size_t)blockIdx.x * G::kPart;
    if (tid < C) out[C * C + tid] = gb;
    if (G::kSlices == 1) {
        if (active) {
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) out[(nn + r * G::Q) * C + kk + c * G::Q] = acc[r][c];
        }
        return;
    }
    __syncthreads();
    float* red = sm;                                              // [kSlices][C * C]
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) red[slice * (C * C) + (nn + r * G::Q) * C + kk + c * G::Q] = acc[r][c];
    __syncthreads();
    for (int e = tid; e < C * C; e += kThreads) {
        float t = red[e];
        for (int sl = 1; sl < G::kSlices; ++sl) t += red[sl * (C * C) + e];
        out[e] = t;
    }
}

// g_W [C*C] and g_b [C]: a warp per element, lanes over blocks in order, fixed butterfly.
__global__ void __launch_bounds__(256)
sum_wgrad(const float* __restrict__ part, int C, int blocks, float* __restrict__ g_w, float* __restrict__ g_b)
{
    const int lane = threadIdx.x & 31, e = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, n = C * C + C;
    if (e >= n) return;
    float s = 0.f;
    for (int k = lane; k < blocks; k += 32) s += part[(size_t)k * n + e];
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
        if (e < C * C) { if (g_w) g_w[e] = s; }
        else if (g_b) g_b[e - C * C] = s;
    }
}

}}}  // namespace esc::fuse::bwd

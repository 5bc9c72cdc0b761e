// Backward pass with the dense large kernel (ESC paper, Section 3.2: LK of 13 x 13 x 16 x 16, output channel n sums over
// every attention input channel k; the dynamic 3x3 kernel stays depth-wise).  With go = dL/dout:
//
//   g_wd[n,k,i,j] = sum_{b,y,x} go[b,n,y,x] * x~[b,k,y+i-6,x+j-6]                         (kernel tap_grad_dense)
//   g_x[b,k]      = sum_n go[b,n] (*) flip(w_dense[n,k]) + go[b,k] (*) flip(dk[b,k]) + g_g[b,k] / (H W)
//
// g_x's first two terms are the forward dense stencil applied to go with the kernel's channel axes swapped and its taps
// rotated by 180 degrees (`flip_dense` prepares it), so they run on the forward kernels; `add_const` adds the third.
// g_dk, g_b, g_W and g_g come from the depth-wise backward's kernels (the 3x3 kernel is depth-wise).
//
// tap_grad_dense: 2 * 16 * 16 * 169 multiply-adds per pixel, on the FP32 pipe.  A persistent block walks tiles of
// 32 x 16 pixels of all images; thread (n, k) keeps the 13 x 13 sums of its channel pair in registers across all its tiles
// and reads, per four pixels of a go row, 13 x 4 16-byte words of x (sixteen columns of thirteen rows) and one of go:
// 676 FMAs per 53 shared-memory reads.  Every block writes its sums once; `sum_dense` adds the blocks in order.
#pragma once
#include "common.cuh"
#include "backward.cuh"

namespace esc { namespace bwd { namespace dense {

constexpr int CA = 16;
constexpr int TX = 32, TY = 16;
constexpr int XW = TX + K - 1, XH = TY + K - 1;       // 44 x 28 staged pixels per channel
constexpr int XPITCH = XW;                            // floats per staged row (a multiple of 4)
constexpr int XPLANE = XH * XPITCH + 4;               // 1236 = 20 mod 32: the eight lanes of a quarter warp read distinct banks
constexpr int GPLANE = TY * TX;
constexpr int kThreads = CA * CA;
constexpr size_t kSmemBytes = (size_t)(CA * XPLANE + CA * GPLANE) * sizeof(float);
constexpr int kPartFloats = CA * CA * TAPS;           // per block
static_assert(XPITCH % 4 == 0 && XPLANE % 4 == 0 && TX % 4 == 0, "16-byte rows");

template <typename T, int LAYOUT>
__global__ void __launch_bounds__(kThreads, 1)
tap_grad_dense(const T* __restrict__ x, const T* __restrict__ go, int B, int C, int H, int W, int tiles_x, int tiles_y,
               float* __restrict__ part)              // [gridDim.x][CA][CA][13][13]
{
    extern __shared__ __align__(16) float sm[];
    float* xs = sm;
    float* gs = sm + CA * XPLANE;
    const int tid = threadIdx.x, k = tid & (CA - 1), n = tid / CA;
    float acc[K][K];
#pragma unroll
    for (int i = 0; i < K; ++i)
#pragma unroll
        for (int j = 0; j < K; ++j) acc[i][j] = 0.f;
    const long long items = (long long)B * tiles_x * tiles_y;
    for (long long it = blockIdx.x; it < items; it += gridDim.x) {
        const int b = (int)(it / ((long long)tiles_x * tiles_y));
        const int tr = (int)(it % ((long long)tiles_x * tiles_y));
        const int y0 = (tr / tiles_x) * TY, x0 = (tr % tiles_x) * TX;
        __syncthreads();                                          // the previous tile is read
        // x with its halo and go, zeros outside the image; the fastest index follows the tensors' layout
        for (int e = tid; e < CA * XH * XW; e += kThreads) {
            int c, r, col;
            if (LAYOUT == kNHWC) { c = e % CA; col = (e / CA) % XW; r = e / (CA * XW); }
            else { col = e % XW; r = (e / XW) % XH; c = e / (XW * XH); }
            const int gy = y0 + r - P, gxx = x0 + col - P;
            float v = 0.f;
            if (gy >= 0 && gy < H && gxx >= 0 && gxx < W) v = Elem<T>::to_f32(x[elem_index<LAYOUT>(b, c, gy, gxx, C, H, W)]);
            xs[c * XPLANE + r * XPITCH + col] = v;
        }
        for (int e = tid; e < CA * TY * TX; e += kThreads) {
            int c, r, col;
            if (LAYOUT == kNHWC) { c = e % CA; col = (e / CA) % TX; r = e / (CA * TX); }
            else { col = e % TX; r = (e / TX) % TY; c = e / (TX * TY); }
            const int gy = y0 + r, gxx = x0 + col;
            float v = 0.f;
            if (gy < H && gxx < W) v = Elem<T>::to_f32(go[elem_index<LAYOUT>(b, c, gy, gxx, C, H, W)]);
            gs[c * GPLANE + r * TX + col] = v;
        }
        __syncthreads();
        const float* xk = xs + k * XPLANE;
        const float* gn = gs + n * GPLANE;
        for (int y = 0; y < TY; ++y)
            for (int xc = 0; xc < TX; xc += 4) {
                const float4 g4 = *reinterpret_cast<const float4*>(gn + y * TX + xc);
#pragma unroll
                for (int i = 0; i < K; ++i) {
                    const float4* row = reinterpret_cast<const float4*>(xk + (y + i) * XPITCH + xc);
                    const float4 a0 = row[0], a1 = row[1], a2 = row[2], a3 = row[3];
                    const float w[16] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w, a2.x, a2.y, a2.z, a2.w, a3.x, a3.y, a3.z, a3.w};
#pragma unroll
                    for (int j = 0; j < K; ++j) {
                        float t = acc[i][j];
                        t = fmaf(g4.x, w[j], t); t = fmaf(g4.y, w[j + 1], t);
                        t = fmaf(g4.z, w[j + 2], t); t = fmaf(g4.w, w[j + 3], t);
                        acc[i][j] = t;
                    }
                }
            }
    }
    float* out = part + ((size_t)blockIdx.x * CA * CA + (size_t)n * CA + k) * TAPS;
#pragma unroll
    for (int i = 0; i < K; ++i)
#pragma unroll
        for (int j = 0; j < K; ++j) out[i * K + j] = acc[i][j];
}

// g_wd [CA][CA][KK][KK] = the middle KK x KK of the blocks' 13 x 13 sums, blocks added in order.
__global__ void __launch_bounds__(256)
sum_dense(const float* __restrict__ part, int blocks, int KK, float* __restrict__ g_wd)
{
    const int e = blockIdx.x * blockDim.x + threadIdx.x, taps = KK * KK, off = (K - KK) / 2;
    if (e >= CA * CA * taps) return;
    const int pair = e / taps, i = (e % taps) / KK + off, j = (e % taps) % KK + off;
    const float* p = part + (size_t)pair * TAPS + i * K + j;
    float s = 0.f;
#pragma unroll 8
    for (int b = 0; b < blocks; ++b) s += p[(size_t)b * kPartFloats];
    g_wd[e] = s;
}

// w_flip[k][n][KK-1-i][KK-1-j] = w_dense[n][k][i][j]
template <typename T>
__global__ void __launch_bounds__(256)
flip_dense(const T* __restrict__ w_dense, int KK, T* __restrict__ w_flip)
{
    const int e = blockIdx.x * blockDim.x + threadIdx.x, taps = KK * KK;
    if (e >= CA * CA * taps) return;
    const int n = e / (CA * taps), k = (e / taps) % CA, t = e % taps;
    w_flip[((size_t)k * CA + n) * taps + (taps - 1 - t)] = w_dense[e];
}

// grad_x[b, c < Ca] += bias[b][c] (the estimator's path), a thread per pixel-channel
template <typename T, int LAYOUT>
__global__ void __launch_bounds__(256)
add_const(T* __restrict__ gx, const float* __restrict__ bias, int B, int C, int Ca, long long HW)
{
    const long long total = (long long)B * Ca * HW;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        long long b, c, q;
        if (LAYOUT == kNHWC) { c = e % Ca; q = (e / Ca) % HW; b = e / (Ca * HW); }
        else { q = e % HW; c = (e / HW) % Ca; b = e / (HW * Ca); }
        const size_t idx = LAYOUT == kNHWC ? ((size_t)b * HW + q) * C + c : ((size_t)b * C + c) * HW + q;
        gx[idx] = Elem<T>::from_f32(Elem<T>::to_f32(gx[idx]) + bias[b * Ca + c]);
    }
}

}}}  // namespace esc::bwd::dense

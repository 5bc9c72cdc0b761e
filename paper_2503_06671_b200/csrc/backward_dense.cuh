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
#include "stencil_toeplitz.cuh"
#include "conv_fuse.cuh"

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

// ---- the same sums on the tensor cores, for bf16 tensors -------------------------------------------------------------
// For one tap (i, j) the sum over pixels is a plain matrix product, go^T [16 channels x pixels] times x shifted by the tap
// [pixels x 16 channels]: every product is useful, bf16 products are exact in fp32 and the accumulation is fp32, so this
// is the FP32 kernel's arithmetic in another order.  Tiles are staged as two planes of eight channels, 16 bytes per pixel
// (any pixel offset is a legal ldmatrix row address; eight consecutive pixels are 128 contiguous bytes: no bank
// conflicts).  Per 16 pixels of a go row a warp loads the A fragments once (ldmatrix.trans: channel x pixel from
// pixel-major storage) and, for each of its taps, the B fragments of x at the shifted position the same way, then two
// mma.sync.m16n8k16 (x channels 0-7, 8-15).  The 169 taps are dealt to the eight warps (22 or 21 each, 8 accumulator
// registers per tap) and stay in registers across all tiles of the block.  NHWC tensors: the next tile is fetched with
// cp.async into a second buffer while this one is multiplied.
namespace mma {
using tma::toep::ldsm_x4_trans; using tma::toep::mma_bf16;
constexpr int kWarps = 8, kThreads = kWarps * 32;
constexpr int kTapsPerWarp = (TAPS + kWarps - 1) / kWarps;          // 22
constexpr int TYM = 8, XHM = TYM + K - 1;                            // tiles of 32 x 8 pixels here: 920 of them at 640x360 balance better over 148 blocks than 460
constexpr int XHALF = XHM * XW * 16;                                 // bytes per plane of eight channels
constexpr int GHALF = TYM * TX * 16;
constexpr int kBufBytes = 2 * XHALF + 2 * GHALF;                      // 36,352 bytes: one tile of x and of go
constexpr size_t kSmemBytes = 2 * (size_t)kBufBytes;                 // two of them
static_assert(TX % 16 == 0, "whole MMA pixel blocks per row");

template <int LAYOUT>
__global__ void __launch_bounds__(kThreads, 1)
tap_grad_dense_bf16(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ go, int B, int C, int H, int W,
                    int tiles_x, int tiles_y, int vec, float* __restrict__ part)   // [gridDim.x][CA][CA][13][13]
{
    extern __shared__ __align__(128) unsigned char smb[];          // two buffers of [x: 2 planes][go: 2 planes]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mi = lane >> 3, mr = lane & 7;      // ldmatrix: lane -> (matrix, row)
    // matrix mi: pixels 8 * (mi >> 1) + mr of the 16, channel half mi & 1
    const uint32_t sm0 = tma::smem_u32(smb);
    const uint32_t x_lane = (uint32_t)((mi & 1) * XHALF + ((mi >> 1) * 8 + mr) * 16);
    const uint32_t g_lane = (uint32_t)(2 * XHALF + (mi & 1) * GHALF + ((mi >> 1) * 8 + mr) * 16);
    uint32_t toff[kTapsPerWarp];                  // byte offset of tap warp + 8 s inside the x tile
#pragma unroll
    for (int s = 0; s < kTapsPerWarp; ++s) {
        const int tap = warp + kWarps * s, i = tap / K, j = tap % K;
        toff[s] = (uint32_t)((i * XW + j) * 16);
    }
    float acc[kTapsPerWarp][2][4];
#pragma unroll
    for (int s = 0; s < kTapsPerWarp; ++s)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[s][h][v] = 0.f;
    const long long items = (long long)B * tiles_x * tiles_y;
    const bool async = LAYOUT == kNHWC && vec != 0;               // a pixel's 16 channels are two aligned 16-byte words
    // NHWC: the next tile is fetched with cp.async (zero fill outside the image) while this one is multiplied
    auto stage_async = [&](long long it, int buf) {
        const int b = (int)(it / ((long long)tiles_x * tiles_y));
        const int tr = (int)(it % ((long long)tiles_x * tiles_y));
        const int y0 = (tr / tiles_x) * TYM, x0 = (tr % tiles_x) * TX;
        const uint32_t xb = sm0 + (uint32_t)(buf * kBufBytes), gb = xb + 2 * XHALF;
        for (int e = tid; e < 2 * XHM * XW; e += kThreads) {
            const int h = e & 1, col = (e >> 1) % XW, r = (e >> 1) / XW;
            const int gy = y0 + r - P, gxx = x0 + col - P;
            const bool valid = gy >= 0 && gy < H && gxx >= 0 && gxx < W;
            fuse::cp_async16(xb + (uint32_t)(h * XHALF + (r * XW + col) * 16),
                             x + (valid ? (((size_t)b * H + gy) * W + gxx) * C + 8 * h : 0), valid);
        }
        for (int e = tid; e < 2 * TYM * TX; e += kThreads) {
            const int h = e & 1, col = (e >> 1) % TX, r = (e >> 1) / TX;
            const int gy = y0 + r, gxx = x0 + col;
            const bool valid = gy < H && gxx < W;
            fuse::cp_async16(gb + (uint32_t)(h * GHALF + (r * TX + col) * 16),
                             go + (valid ? (((size_t)b * H + gy) * W + gxx) * C + 8 * h : 0), valid);
        }
        fuse::cp_async_commit();
    };
    auto stage_sync = [&](long long it) {                         // any layout: element by element into buffer 0
        const int b = (int)(it / ((long long)tiles_x * tiles_y));
        const int tr = (int)(it % ((long long)tiles_x * tiles_y));
        const int y0 = (tr / tiles_x) * TYM, x0 = (tr % tiles_x) * TX;
        unsigned char* xs = smb;
        unsigned char* gs = smb + 2 * XHALF;
        const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
        for (int e = tid; e < CA * XHM * XW; e += kThreads) {
            int c, r, col;
            if (LAYOUT == kNHWC) { c = e % CA; col = (e / CA) % XW; r = e / (CA * XW); }
            else { col = e % XW; r = (e / XW) % XHM; c = e / (XW * XHM); }
            const int gy = y0 + r - P, gxx = x0 + col - P;
            __nv_bfloat16 v = zero;
            if (gy >= 0 && gy < H && gxx >= 0 && gxx < W) v = x[elem_index<LAYOUT>(b, c, gy, gxx, C, H, W)];
            *reinterpret_cast<__nv_bfloat16*>(xs + (c >> 3) * XHALF + (r * XW + col) * 16 + (c & 7) * 2) = v;
        }
        for (int e = tid; e < CA * TYM * TX; e += kThreads) {
            int c, r, col;
            if (LAYOUT == kNHWC) { c = e % CA; col = (e / CA) % TX; r = e / (CA * TX); }
            else { col = e % TX; r = (e / TX) % TYM; c = e / (TX * TYM); }
            const int gy = y0 + r, gxx = x0 + col;
            __nv_bfloat16 v = zero;
            if (gy < H && gxx < W) v = go[elem_index<LAYOUT>(b, c, gy, gxx, C, H, W)];
            *reinterpret_cast<__nv_bfloat16*>(gs + (c >> 3) * GHALF + (r * TX + col) * 16 + (c & 7) * 2) = v;
        }
    };
    if (async && (long long)blockIdx.x < items) stage_async(blockIdx.x, 0);
    int k = 0;
    for (long long it = blockIdx.x; it < items; it += gridDim.x, ++k) {
        const int buf = async ? (k & 1) : 0;
        if (async) {
            const long long nx = it + gridDim.x;
            if (nx < items) stage_async(nx, buf ^ 1);
            else fuse::cp_async_commit();
            fuse::cp_async_wait<1>();
        } else {
            __syncthreads();                                      // the previous tile is read
            stage_sync(it);
        }
        __syncthreads();                                          // the tile is there for every warp
        const uint32_t base = sm0 + (uint32_t)(buf * kBufBytes);
        for (int y = 0; y < TYM; ++y)
#pragma unroll 1
            for (int xb = 0; xb < TX / 16; ++xb) {
                uint32_t a[4];                                    // go: (channels 0-7 | 8-15) x (pixels 0-7 | 8-15)
                ldsm_x4_trans(base + g_lane + (uint32_t)((y * TX + xb * 16) * 16), a);
                const uint32_t xrow = base + x_lane + (uint32_t)((y * XW + xb * 16) * 16);
#pragma unroll
                for (int s = 0; s < kTapsPerWarp; ++s) {
                    if (s < kTapsPerWarp - 1 || warp + kWarps * s < TAPS) {
                        uint32_t bf[4];                           // x at the tap's offset: same arrangement
                        ldsm_x4_trans(xrow + toff[s], bf);
                        mma_bf16(acc[s][0], a[0], a[1], a[2], a[3], bf[0], bf[2]);
                        mma_bf16(acc[s][1], a[0], a[1], a[2], a[3], bf[1], bf[3]);
                    }
                }
            }
        if (async) __syncthreads();                               // this buffer may be refilled
    }
    if (async) fuse::cp_async_wait<0>();
    // acc[s][h]: [0], [1] = go channel g, x channels 8 h + 2t, + 1; [2], [3] = go channel g + 8
    const int g = lane >> 2, t = lane & 3;
    float* out = part + (size_t)blockIdx.x * kPartFloats;
#pragma unroll
    for (int s = 0; s < kTapsPerWarp; ++s) {
        const int tap = warp + kWarps * s;
        if (tap < TAPS) {
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const int n = g + 8 * (v >> 1), k = 8 * h + 2 * t + (v & 1);
                    out[((size_t)n * CA + k) * TAPS + tap] = acc[s][h][v];
                }
        }
    }
}
}  // namespace mma

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

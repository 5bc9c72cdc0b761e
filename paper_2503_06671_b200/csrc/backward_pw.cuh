// Backward pass of the decomposed form (ESC paper, Eq. 5): the point-wise filter LK^c (a bias-free 1x1 convolution P over
// the C_a attention channels) in front of the depth-wise stage.  With m = P x_att (the mixed features), dk from the GAP
// of the UNMIXED features and g_m = dL/dm:
//
//   g_tap, g_lk, g_dk, g_b, g_W, g_g      as for the depth-wise form, with m in the place of x_att -- except the mean
//                                         that g_W multiplies, which stays the mean of x_att
//   g_m[b,n]  = go[b,n] (*) flip(LK[n] + ZP(dk[b,n]))                      (the forward stencil with rotated kernels)
//   g_P[n,k]  = sum_{b,pixels} g_m[b,n] x[b,k]
//   g_x[b,k]  = sum_n P[n,k] g_m[b,n] + g_g[b,k] / (H W)
//
// so the pass is the depth-wise one between two per-pixel kernels of this file: `mix` writes m into the attention
// channels of grad_x (where the tap-gradient kernels read it as their "x") and the per-chunk sums of x_att; `back`
// turns the g_m that the stencil pass has left in grad_x into g_x in place and forms per-chunk partial sums of g_P.
// m and g_m are stored in the tensors' element type, as every feature map of the network is.  All sums are taken in
// a fixed order.
#pragma once
#include "common.cuh"
#include "backward.cuh"

namespace esc { namespace bwd { namespace pw {

constexpr int kThreads = 256;                 // one pixel per thread and pass
constexpr int kPasses = 2;
constexpr int kChunk = kThreads * kPasses;    // pixels of one image per block
constexpr int kPitch = kThreads + 4;          // floats per staged channel row (16-byte rows, banks shifted by four)

inline int chunks_of(long long HW) { return (int)((HW + kChunk - 1) / kChunk); }
inline bool supported(int Ca) { return Ca == 4 || Ca == 8 || Ca == 16 || Ca == 32; }

template <typename T> __device__ __forceinline__ uint4 pack16(const float* f);
template <> __device__ __forceinline__ uint4 pack16<float>(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
template <> __device__ __forceinline__ uint4 pack16<__nv_bfloat16>(const float* f) {
    uint4 v;
    __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]), b = __floats2bfloat162_rn(f[2], f[3]);
    __nv_bfloat162 c = __floats2bfloat162_rn(f[4], f[5]), d = __floats2bfloat162_rn(f[6], f[7]);
    v.x = *reinterpret_cast<unsigned*>(&a); v.y = *reinterpret_cast<unsigned*>(&b);
    v.z = *reinterpret_cast<unsigned*>(&c); v.w = *reinterpret_cast<unsigned*>(&d);
    return v;
}

// The CA attention values of pixel q of image b, widened to fp32.  `vec`: NHWC with 16-byte aligned pixel rows.
template <typename T, int LAYOUT, int CA>
__device__ __forceinline__ void load_px(const T* __restrict__ t, size_t b, int C, size_t HW, size_t q, bool vec, float (&v)[CA]) {
    constexpr int V = Elem<T>::kVec;
    if (LAYOUT == kNHWC) {
        const T* p = t + (b * HW + q) * C;
        if (CA % V == 0 && vec) {
#pragma unroll
            for (int k = 0; k < CA / V * V; k += V) unpack16<T>(*reinterpret_cast<const uint4*>(p + k), &v[k]);
        } else {
#pragma unroll
            for (int k = 0; k < CA; ++k) v[k] = Elem<T>::to_f32(p[k]);
        }
    } else {
#pragma unroll
        for (int k = 0; k < CA; ++k) v[k] = Elem<T>::to_f32(t[(b * C + k) * HW + q]);
    }
}
// Channels k0 .. k0+G-1 of one pixel (G = 8, or 4 where C_a = 4; k0 a multiple of G).
template <typename T, int LAYOUT, int G>
__device__ __forceinline__ void store_group(T* __restrict__ t, size_t b, int C, size_t HW, size_t q, bool vec, int k0, const float (&v)[G]) {
    constexpr int V = Elem<T>::kVec;
    if (LAYOUT == kNHWC) {
        T* p = t + (b * HW + q) * C + k0;
        if (G % V == 0 && vec) {
#pragma unroll
            for (int k = 0; k < G / V * V; k += V) *reinterpret_cast<uint4*>(p + k) = pack16<T>(&v[k]);
        } else {
#pragma unroll
            for (int k = 0; k < G; ++k) p[k] = Elem<T>::from_f32(v[k]);
        }
    } else {
#pragma unroll
        for (int k = 0; k < G; ++k) t[(b * C + k0 + k) * HW + q] = Elem<T>::from_f32(v[k]);
    }
}

// ---- m = P x_att into the attention channels of `m`; per-chunk sums of x_att -------------------------------------
// Block = (image, chunk of kChunk pixels).  P sits in shared memory (read as broadcast 16-byte rows), a pixel's
// channels in registers.
template <typename T, int LAYOUT, int CA>
__global__ void __launch_bounds__(kThreads, CA <= 16 ? 4 : 2)
mix(const T* __restrict__ x, const T* __restrict__ w_point, T* __restrict__ m, int C, long long HW_, int chunks, int vec_,
    float* __restrict__ xs_part)              // [B][chunks][CA]
{
    __shared__ __align__(16) float ps[CA * CA];
    __shared__ float red[kThreads / 32][CA];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t HW = (size_t)HW_, b = blockIdx.x / chunks;
    const int ch = blockIdx.x % chunks;
    const bool vec = vec_ != 0;
    for (int e = tid; e < CA * CA; e += kThreads) ps[e] = Elem<T>::to_f32(w_point[e]);
    __syncthreads();
    float sx[CA];
#pragma unroll
    for (int k = 0; k < CA; ++k) sx[k] = 0.f;
    for (int pass = 0; pass < kPasses; ++pass) {
        const size_t q = (size_t)ch * kChunk + (size_t)pass * kThreads + tid;
        if (q >= HW) break;
        float v[CA];
        load_px<T, LAYOUT, CA>(x, b, C, HW, q, vec, v);
#pragma unroll
        for (int k = 0; k < CA; ++k) sx[k] += v[k];
        // a group of outputs at a time, stored at once: a rolled loop, so that P is not read ahead into a hundred registers
        constexpr int G = CA >= 8 ? 8 : 4;
#pragma unroll 1
        for (int n0 = 0; n0 < CA; n0 += G) {
            float o[G];
#pragma unroll
            for (int j = 0; j < G; ++j) {
                float s = 0.f;
#pragma unroll
                for (int k = 0; k < CA; ++k) s = fmaf(ps[(n0 + j) * CA + k], v[k], s);
                o[j] = s;
            }
            store_group<T, LAYOUT, G>(m, b, C, HW, q, vec, n0, o);
        }
    }
#pragma unroll
    for (int k = 0; k < CA; ++k) {
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) sx[k] += __shfl_xor_sync(0xffffffffu, sx[k], o);
        if (lane == 0) red[warp][k] = sx[k];
    }
    __syncthreads();
    if (tid < CA) {
        float s = red[0][tid];
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) s += red[w][tid];
        xs_part[((size_t)b * chunks + ch) * CA + tid] = s;
    }
}

// ---- sum of x_att per (image, channel) into the tap-gradient table's slot for it ------------------------------------
// A warp per (image, channel): lanes take every 32nd chunk in order, then a fixed butterfly.
__global__ void __launch_bounds__(256)
sum_x(const float* __restrict__ xs_part, int BCa, int Ca, int chunks, float* __restrict__ gtap)
{
    const int lane = threadIdx.x & 31, e = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (e >= BCa) return;
    const int b = e / Ca, k = e % Ca;
    float s = 0.f;
    for (int c = lane; c < chunks; c += 32) s += xs_part[((size_t)b * chunks + c) * Ca + k];
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) gtap[(size_t)e * kSlot + TAPS] = s;
}

// ---- g_x = P^T g_m + constant, in place; per-chunk partial sums of g_P ---------------------------------------------
// Block = (image, chunk).  Per pass a thread turns its pixel's g_m into g_x (P's rows broadcast from shared memory) and
// stages g_m and x_att of the pass channel-major.  The outer products g_m[n] x[k] are then register-tiled: the CA x CA
// pairs are cut into 4x4 tiles, the pass's 256 pixels into `kSlices` interleaved slices, thread (tile, slice) reads
// four pixels of its four g_m rows and four x rows at a time (eight 16-byte reads per 64 FMAs; lanes of a slice group
// read adjacent 16-byte words).  At the end the slices' sums are added per pair in slice order.
// Dynamic shared memory: P [CA][CA] | constants [CA] | g_m [CA][kPitch] | x [CA][kPitch]  (re-used for the slices' sums).
template <int CA> struct BackGeom {
    static constexpr int kTiles = CA * CA / 16;                 // 4x4 tiles of (n, k) pairs
    static constexpr int kSlices = kThreads / kTiles;           // pixel slices per pass
    static constexpr int kPx = kThreads / kSlices;              // pixels per slice and pass
    static constexpr int kStage = 2 * CA * kPitch > kSlices * CA * CA ? 2 * CA * kPitch : kSlices * CA * CA;
    static_assert(CA % 4 == 0 && kTiles >= 1 && kTiles <= kThreads && kThreads % kTiles == 0, "tiling");
};
template <int CA> constexpr size_t back_smem_bytes() { return (size_t)(CA * CA + CA + BackGeom<CA>::kStage) * sizeof(float); }

template <typename T, int LAYOUT, int CA>
__global__ void __launch_bounds__(kThreads, CA <= 16 ? 3 : 2)
back(const T* __restrict__ x, const T* __restrict__ w_point, T* __restrict__ gx, const float* __restrict__ bias, int C,
     long long HW_, int chunks, int vec_, float* __restrict__ gp_part)          // [B * chunks][CA * CA]
{
    using G = BackGeom<CA>;
    extern __shared__ __align__(16) float sm[];
    float* ps = sm;
    float* bs = ps + CA * CA;
    float* gs = bs + CA;
    float* xs = gs + CA * kPitch;
    const int tid = threadIdx.x;
    const size_t HW = (size_t)HW_, b = blockIdx.x / chunks;
    const int ch = blockIdx.x % chunks;
    const bool vec = vec_ != 0;
    const int tile = tid / G::kSlices, slice = tid % G::kSlices;
    const int n0 = (tile / (CA / 4)) * 4, k0 = (tile % (CA / 4)) * 4;
    for (int e = tid; e < CA * CA; e += kThreads) ps[e] = Elem<T>::to_f32(w_point[e]);
    if (tid < CA) bs[tid] = bias[b * CA + tid];
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int pass = 0; pass < kPasses; ++pass) {
        const size_t q0 = (size_t)ch * kChunk + (size_t)pass * kThreads;
        if (q0 >= HW) break;
        const size_t q = q0 + tid;
        __syncthreads();                                         // P and the constants are there; the last pass's staged rows are read
        {
            float gm[CA];
            {
                float xv[CA];
                if (q < HW) {
                    load_px<T, LAYOUT, CA>(gx, b, C, HW, q, vec, gm);
                    load_px<T, LAYOUT, CA>(x, b, C, HW, q, vec, xv);
                } else {
#pragma unroll
                    for (int k = 0; k < CA; ++k) gm[k] = xv[k] = 0.f;
                }
#pragma unroll
                for (int k = 0; k < CA; ++k) {
                    gs[k * kPitch + tid] = gm[k];
                    xs[k * kPitch + tid] = xv[k];
                }
            }
            if (q < HW) {
                // a group of channels at a time (rolled, as in `mix`)
                constexpr int G = CA >= 8 ? 8 : 4;
#pragma unroll 1
                for (int k0 = 0; k0 < CA; k0 += G) {
                    float o[G];
#pragma unroll
                    for (int j = 0; j < G; ++j) o[j] = bs[k0 + j];
#pragma unroll
                    for (int n = 0; n < CA; ++n)
#pragma unroll
                        for (int j = 0; j < G; ++j) o[j] = fmaf(ps[n * CA + k0 + j], gm[n], o[j]);
                    store_group<T, LAYOUT, G>(gx, b, C, HW, q, vec, k0, o);
                }
            }
        }
        __syncthreads();
        if (G::kPx >= 4) {
            // pixels slice*4 + i*(4*kSlices) .. +3
#pragma unroll 2
            for (int i = 0; i < G::kPx / 4; ++i) {
                const int px = slice * 4 + i * 4 * G::kSlices;
                float4 u[4], w[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    u[r] = *reinterpret_cast<const float4*>(gs + (n0 + r) * kPitch + px);
                    w[r] = *reinterpret_cast<const float4*>(xs + (k0 + r) * kPitch + px);
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
        } else {
            // fewer than four pixels per slice (C_a = 4: one tile, a pixel per thread)
#pragma unroll
            for (int i = 0; i < G::kPx; ++i) {
                const int px = slice * G::kPx + i;
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(gs[(n0 + r) * kPitch + px], xs[(k0 + c) * kPitch + px], acc[r][c]);
            }
        }
    }
    __syncthreads();
    float* red = gs;                                             // [kSlices][CA * CA]
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) red[slice * (CA * CA) + (n0 + r) * CA + k0 + c] = acc[r][c];
    __syncthreads();
    for (int e = tid; e < CA * CA; e += kThreads) {
        float t = red[e];
        for (int sl = 1; sl < G::kSlices; ++sl) t += red[sl * (CA * CA) + e];
        gp_part[(size_t)blockIdx.x * (CA * CA) + e] = t;
    }
}

// ---- g_P[e] = sum over blocks of the partial sums: a warp per element, lanes over blocks in order, butterfly ---------
__global__ void __launch_bounds__(256)
sum_gp(const float* __restrict__ gp_part, int elems, int blocks, float* __restrict__ g_wp)
{
    const int lane = threadIdx.x & 31, e = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (e >= elems) return;
    float s = 0.f;
    for (int k = lane; k < blocks; k += 32) s += gp_part[(size_t)k * elems + e];
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) g_wp[e] = s;
}

}}}  // namespace esc::bwd::pw

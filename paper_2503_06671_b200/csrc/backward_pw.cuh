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
constexpr int kPasses = 4;
constexpr int kChunk = kThreads * kPasses;    // pixels of one image per block
constexpr int kPitch = kThreads + 4;          // floats per staged channel row (16-byte rows, banks shifted by four)

inline int chunks_of(long long HW) { return (int)((HW + kChunk - 1) / kChunk); }
inline bool supported(int Ca) { return Ca == 4 || Ca == 8 || Ca == 16 || Ca == 32; }
template <int CA> constexpr size_t back_smem_bytes() { return (size_t)(CA * CA + CA + 2 * CA * kPitch) * sizeof(float); }

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
template <typename T, int LAYOUT, int CA>
__device__ __forceinline__ void store_px(T* __restrict__ t, size_t b, int C, size_t HW, size_t q, bool vec, const float (&v)[CA]) {
    constexpr int V = Elem<T>::kVec;
    if (LAYOUT == kNHWC) {
        T* p = t + (b * HW + q) * C;
        if (CA % V == 0 && vec) {
#pragma unroll
            for (int k = 0; k < CA / V * V; k += V) *reinterpret_cast<uint4*>(p + k) = pack16<T>(&v[k]);
        } else {
#pragma unroll
            for (int k = 0; k < CA; ++k) p[k] = Elem<T>::from_f32(v[k]);
        }
    } else {
#pragma unroll
        for (int k = 0; k < CA; ++k) t[(b * C + k) * HW + q] = Elem<T>::from_f32(v[k]);
    }
}

// ---- m = P x_att into the attention channels of `m`; per-chunk sums of x_att -------------------------------------
// Block = (image, chunk of kChunk pixels).  P sits in shared memory (read as broadcast 16-byte rows), a pixel's
// channels in registers.
template <typename T, int LAYOUT, int CA>
__global__ void __launch_bounds__(kThreads)
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
        float v[CA], o[CA];
        load_px<T, LAYOUT, CA>(x, b, C, HW, q, vec, v);
#pragma unroll
        for (int k = 0; k < CA; ++k) sx[k] += v[k];
#pragma unroll
        for (int n = 0; n < CA; ++n) {
            float s = 0.f;
#pragma unroll
            for (int k = 0; k < CA; ++k) s = fmaf(ps[n * CA + k], v[k], s);
            o[n] = s;
        }
        store_px<T, LAYOUT, CA>(m, b, C, HW, q, vec, o);
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
// stages g_m and x_att of the pass channel-major; then thread (n, k) adds the pass's 256 products g_m[n] x[k].
// Dynamic shared memory: P [CA][CA] | constants [CA] | g_m [CA][kPitch] | x [CA][kPitch].
template <typename T, int LAYOUT, int CA>
__global__ void __launch_bounds__(kThreads)
back(const T* __restrict__ x, const T* __restrict__ w_point, T* __restrict__ gx, const float* __restrict__ bias, int C,
     long long HW_, int chunks, int vec_, float* __restrict__ gp_part)          // [B * chunks][CA * CA]
{
    extern __shared__ __align__(16) float sm[];
    float* ps = sm;
    float* bs = ps + CA * CA;
    float* gs = bs + CA;
    float* xs = gs + CA * kPitch;
    constexpr int NP = (CA * CA + kThreads - 1) / kThreads;     // (n, k) pairs per thread
    const int tid = threadIdx.x;
    const size_t HW = (size_t)HW_, b = blockIdx.x / chunks;
    const int ch = blockIdx.x % chunks;
    const bool vec = vec_ != 0;
    for (int e = tid; e < CA * CA; e += kThreads) ps[e] = Elem<T>::to_f32(w_point[e]);
    if (tid < CA) bs[tid] = bias[b * CA + tid];
    float acc[NP];
#pragma unroll
    for (int e = 0; e < NP; ++e) acc[e] = 0.f;
    for (int pass = 0; pass < kPasses; ++pass) {
        const size_t q0 = (size_t)ch * kChunk + (size_t)pass * kThreads;
        if (q0 >= HW) break;
        const size_t q = q0 + tid;
        __syncthreads();                                         // P and the constants are there; the last pass's staged rows are read
        float gm[CA], xv[CA];
        if (q < HW) {
            load_px<T, LAYOUT, CA>(gx, b, C, HW, q, vec, gm);
            load_px<T, LAYOUT, CA>(x, b, C, HW, q, vec, xv);
            float o[CA];
#pragma unroll
            for (int k = 0; k < CA; ++k) o[k] = bs[k];
#pragma unroll
            for (int n = 0; n < CA; ++n)
#pragma unroll
                for (int k = 0; k < CA; ++k) o[k] = fmaf(ps[n * CA + k], gm[n], o[k]);
            store_px<T, LAYOUT, CA>(gx, b, C, HW, q, vec, o);
        } else {
#pragma unroll
            for (int k = 0; k < CA; ++k) gm[k] = xv[k] = 0.f;
        }
#pragma unroll
        for (int k = 0; k < CA; ++k) {
            gs[k * kPitch + tid] = gm[k];
            xs[k * kPitch + tid] = xv[k];
        }
        __syncthreads();
#pragma unroll
        for (int e = 0; e < NP; ++e) {
            const int pair = e * kThreads + tid;
            if (pair < CA * CA) {
                const float4* a = reinterpret_cast<const float4*>(gs + (pair / CA) * kPitch);
                const float4* c = reinterpret_cast<const float4*>(xs + (pair % CA) * kPitch);
                float s = acc[e];
#pragma unroll 4
                for (int i = 0; i < kThreads / 4; ++i) {
                    const float4 u = a[i], w = c[i];
                    s = fmaf(u.x, w.x, s); s = fmaf(u.y, w.y, s); s = fmaf(u.z, w.z, s); s = fmaf(u.w, w.w, s);
                }
                acc[e] = s;
            }
        }
    }
#pragma unroll
    for (int e = 0; e < NP; ++e) {
        const int pair = e * kThreads + tid;
        if (pair < CA * CA) gp_part[(size_t)blockIdx.x * (CA * CA) + pair] = acc[e];
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

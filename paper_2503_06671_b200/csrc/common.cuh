// Shared device helpers for the ConvAttn kernels (ESC paper, Section 3.3, Eq. 4).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace esc {

constexpr int kNCHW = 0;
constexpr int kNHWC = 1;

// Control words at the start of a workspace (all 32-bit).
//   [0]            status word (ESC_OK or ESC_DEV_TIMEOUT)
//   [1]            debug word (where a wait gave up)
//   [2..3]         reserved
//   [4 .. 4+B)     per-image arrival counters of the GAP kernel
constexpr int kCtrlHeaderWords = 4;
constexpr int kMaxSlabs = 512;         // upper bound on GAP partial sums per image
constexpr unsigned kDevTimeout = 8;    // == ESC_DEV_TIMEOUT

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kVec = 4;  // elements per 16-byte vector
    __device__ static __forceinline__ float to_f32(float v) { return v; }
    __device__ static __forceinline__ float from_f32(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kVec = 8;
    __device__ static __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
    __device__ static __forceinline__ __nv_bfloat16 from_f32(float v) { return __float2bfloat16_rn(v); }
};

// Element index of logical (b,c,y,x) in a dense tensor of the given layout.
template <int LAYOUT>
__device__ __forceinline__ size_t elem_index(int b, int c, int y, int x, int C, int H, int W) {
    if (LAYOUT == kNCHW) return (((size_t)b * C + c) * H + y) * (size_t)W + x;
    return (((size_t)b * H + y) * (size_t)W + x) * C + c;
}

// 16-byte vector of T widened to fp32.
template <typename T> __device__ __forceinline__ void unpack16(const uint4& v, float* f);
template <> __device__ __forceinline__ void unpack16<float>(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
template <> __device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4& v, float* f) {
    // bf16 -> fp32 is a 16-bit shift: the low half of each word is the even element.
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Programmatic dependent launch (PTX griddepcontrol): the producer lets the next kernel in the
// stream start early; the consumer blocks until the producer grid has finished and its writes
// are visible.  Both are no-ops when the kernel was launched without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_primary() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

}  // namespace esc

// The module's closing step (ESC paper, Section 3.3, Eq. 4 line 4): F_fuse = Conv_fuse(Concat(F_res, F_idt)), a
// 1x1 convolution over all C channels with bias, plus the residual connection of the ESC block around the module
// (Eq. 3 line 3):
//
//   out[b,n,y,x] = b_fuse[n] + sum_c w_fuse[n,c] * cat[b,c,y,x]  ( + residual[b,n,y,x] ),   cat = (F_res | F_idt)
//
// conv_fuse_nhwc_bf16: NHWC bf16, C a multiple of 16 up to 128.  A pixel's C channels are the K dimension of a
// small GEMM (M = pixels, N = K = C) on the tensor cores (mma.sync bf16, fp32 accumulation).  The concatenation is
// never materialised: the attention channels F_res are read from `att` (where the stencil kernel has written
// them, the first C_a channels of each pixel of the output tensor) and the identity channels straight from x, so
// the stencil kernel need not copy them; a block stages 64 pixels, multiplies, and writes whole 2C-byte pixels
// over the same 64 pixels of `out` -- in place, which is safe because a block reads its pixels before it
// writes them and no other block touches them.
// conv_fuse_generic: any type and layout, one block per 32 pixels, cat read from `out` in place.
#pragma once
#include "common.cuh"
#include "stencil_toeplitz.cuh"

namespace esc { namespace fuse {

constexpr int kPix = 64, kThreads = 128;      // pixels per block: four warps of 16 pixels

struct Params {
    const __nv_bfloat16* att;         // tensor whose first Ca channels per pixel are F_res (pixel pitch C)
    const __nv_bfloat16* idt;         // tensor whose channels Ca .. C-1 per pixel are F_idt (pixel pitch C)
    const __nv_bfloat16* w;           // [C][C], row = output channel
    const __nv_bfloat16* bias;        // [C] or nullptr
    const __nv_bfloat16* residual;    // [pixels][C] or nullptr
    __nv_bfloat16* out;               // [pixels][C]
    long long pixels;
    int C, Ca;
};

template <int C>
__global__ void __launch_bounds__(kThreads)
conv_fuse_nhwc_bf16(const Params p)
{
    constexpr int PITCH = C * 2 + 16;                       // bytes per staged row: 16-byte rows of an ldmatrix fall in different banks
    constexpr int NT = C / 8, KS = C / 16;
    extern __shared__ __align__(16) unsigned char smem[];
    unsigned char* wsm = smem;                              // [C][PITCH]: w_fuse, row n = output channel
    unsigned char* xsm = smem + C * PITCH;                  // [kPix][PITCH]: cat of the tile's pixels; later the results
    unsigned char* rsm = xsm + kPix * PITCH;                // [kPix][PITCH]: the residual of the same pixels
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;

    // ---- stage w_fuse and the 64 pixels (16-byte pieces; channels below Ca from `att`, the rest from `idt`) -----
    constexpr int CH = C / 8;                               // 16-byte pieces per row
    for (int e = tid; e < C * CH; e += kThreads) {
        const int r = e / CH, q = e % CH;
        *reinterpret_cast<uint4*>(wsm + r * PITCH + q * 16) = __ldg(reinterpret_cast<const uint4*>(p.w + (size_t)r * C) + q);
    }
    // a block keeps w_fuse and walks tiles of 64 pixels
    const long long ntiles = (p.pixels + kPix - 1) / kPix;
    for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const long long px0 = tile * kPix;
    for (int e = tid; e < kPix * CH; e += kThreads) {
        const int r = e / CH, q = e % CH;
        const long long px = px0 + r;
        uint4 v = make_uint4(0u, 0u, 0u, 0u), rv = make_uint4(0u, 0u, 0u, 0u);
        if (px < p.pixels) {
            const __nv_bfloat16* src = (q * 8 < p.Ca ? p.att : p.idt) + (size_t)px * C;
            v = __ldcg(reinterpret_cast<const uint4*>(src) + q);
            if (p.residual) rv = __ldcg(reinterpret_cast<const uint4*>(p.residual + (size_t)px * C) + q);
        }
        *reinterpret_cast<uint4*>(xsm + r * PITCH + q * 16) = v;
        *reinterpret_cast<uint4*>(rsm + r * PITCH + q * 16) = rv;
    }
    __syncthreads();

    // ---- D (16 pixels x C) = A (16 x C) x B (C x C) per warp ------------------------------------------------
    float acc[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[n][v] = 0.f;
    const int mi = lane >> 3, mr = lane & 7;
    const uint32_t a_lane = tma::smem_u32(xsm) + (uint32_t)((warp * 16 + (mi & 1) * 8 + mr) * PITCH + (mi >> 1) * 16);
    const uint32_t b_lane = tma::smem_u32(wsm) + (uint32_t)(((mi >> 1) * 8 + mr) * PITCH + (mi & 1) * 16);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        uint32_t a[4];
        tma::toep::ldsm_x4(a_lane + ks * 32, a);            // rows 0-7 / 8-15 of the warp's pixels, k halves 0 / 1
#pragma unroll
        for (int n2 = 0; n2 < NT / 2; ++n2) {
            uint32_t b[4];                                  // output channels 16 n2 .. + 7 (k halves), then + 8 .. + 15
            tma::toep::ldsm_x4(b_lane + (uint32_t)(n2 * 16 * PITCH) + ks * 32, b);
            tma::toep::mma_bf16(acc[2 * n2], a[0], a[1], a[2], a[3], b[0], b[1]);
            tma::toep::mma_bf16(acc[2 * n2 + 1], a[0], a[1], a[2], a[3], b[2], b[3]);
        }
    }
    __syncthreads();                                        // everybody has read the staged pixels

    // ---- bias and residual are added in fp32; one rounding to bf16; results staged over the block's pixels -------
    // acc[n]: [0], [1] = pixel g, output channels 8n + 2t, + 1; [2], [3] = pixel g + 8
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        const int oc = 8 * n + 2 * t;
        float b0 = 0.f, b1 = 0.f;
        if (p.bias) { b0 = __bfloat162float(p.bias[oc]); b1 = __bfloat162float(p.bias[oc + 1]); }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int r = warp * 16 + g + 8 * h;
            float v0 = acc[n][2 * h] + b0, v1 = acc[n][2 * h + 1] + b1;
            const uint32_t rr = *reinterpret_cast<const uint32_t*>(rsm + r * PITCH + oc * 2);   // zero without a residual
            v0 += __uint_as_float(rr << 16);
            v1 += __uint_as_float(rr & 0xffff0000u);
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
            *reinterpret_cast<uint32_t*>(xsm + r * PITCH + oc * 2) = *reinterpret_cast<const uint32_t*>(&h2);
        }
    }
    __syncthreads();
    for (int e = tid; e < kPix * CH; e += kThreads) {
        const int r = e / CH, q = e % CH;
        const long long px = px0 + r;
        if (px < p.pixels)
            *(reinterpret_cast<uint4*>(p.out + (size_t)px * C) + q) = *reinterpret_cast<const uint4*>(xsm + r * PITCH + q * 16);
    }
    __syncthreads();                                        // the staging areas are re-used by the next tile
    }
}

// Any type and layout: a block takes 32 pixels, reads their C values of `out` (the concatenated map written by the
// stages before) into shared memory as fp32, then every thread computes outputs (pixel, channel) and writes them
// back to the same pixels.
constexpr int kGenPix = 32, kGenThreads = 256;
template <typename T, int LAYOUT>
__global__ void __launch_bounds__(kGenThreads)
conv_fuse_generic(T* __restrict__ out, const T* __restrict__ w, const T* __restrict__ bias, const T* __restrict__ residual,
                  int B, int C, int H, int W)
{
    extern __shared__ float cat[];                          // [kGenPix][C]
    const long long HW = (long long)H * W, pixels = (long long)B * HW, px0 = (long long)blockIdx.x * kGenPix;
    auto index = [&](long long px, int c) -> size_t {
        const long long b = px / HW, r = px - b * HW;
        return LAYOUT == kNCHW ? ((size_t)b * C + c) * HW + r : (size_t)px * C + c;
    };
    for (int e = threadIdx.x; e < kGenPix * C; e += kGenThreads) {
        const int r = LAYOUT == kNCHW ? e % kGenPix : e / C, c = LAYOUT == kNCHW ? e / kGenPix : e % C;
        const long long px = px0 + r;
        cat[r * C + c] = px < pixels ? Elem<T>::to_f32(out[index(px, c)]) : 0.f;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < kGenPix * C; e += kGenThreads) {
        const int r = LAYOUT == kNCHW ? e % kGenPix : e / C, n = LAYOUT == kNCHW ? e / kGenPix : e % C;
        const long long px = px0 + r;
        if (px >= pixels) continue;
        float s = bias ? Elem<T>::to_f32(bias[n]) : 0.f;
        const T* wr = w + (size_t)n * C;
        const float* v = cat + r * C;
        for (int c = 0; c < C; ++c) s = fmaf(Elem<T>::to_f32(wr[c]), v[c], s);
        if (residual) s += Elem<T>::to_f32(residual[index(px, n)]);
        out[index(px, n)] = Elem<T>::from_f32(s);
    }
}

inline bool fast_applies(int C, int Ca, int dtype, int layout) {
    return dtype == 1 /*bf16*/ && layout == kNHWC && (C == 32 || C == 48 || C == 64 || C == 96 || C == 128) && Ca % 8 == 0;
}

template <int C>
inline cudaError_t launch_fast_c(const Params& p, cudaStream_t st) {
    constexpr int PITCH = C * 2 + 16;
    const size_t smem = (size_t)(C + 2 * kPix) * PITCH;
    static bool attr_set[tma::kMaxDevices] = {};
    const int dev = tma::current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (!attr_set[dev] && smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(conv_fuse_nhwc_bf16<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const long long ntiles = (p.pixels + kPix - 1) / kPix, cap = 8LL * (tma::sm_count() > 0 ? tma::sm_count() : 148);
    conv_fuse_nhwc_bf16<C><<<(unsigned)(ntiles < cap ? ntiles : cap), kThreads, smem, st>>>(p);
    return cudaGetLastError();
}

inline cudaError_t launch_fast(const Params& p, cudaStream_t st) {
    switch (p.C) {
        case 32: return launch_fast_c<32>(p, st);
        case 48: return launch_fast_c<48>(p, st);
        case 64: return launch_fast_c<64>(p, st);
        case 96: return launch_fast_c<96>(p, st);
        case 128: return launch_fast_c<128>(p, st);
        default: return cudaErrorInvalidValue;
    }
}

}}  // namespace esc::fuse

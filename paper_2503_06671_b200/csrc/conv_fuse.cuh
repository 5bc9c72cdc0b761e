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
#include "stencil_toeplitz_nchw.cuh"

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

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    // 16 bytes global -> shared without a register in between; an invalid piece is zero-filled (source size 0)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
template <int C> struct Stages { static constexpr int N = C <= 64 ? 3 : 2; };   // tiles resident per block (one worked on, the rest in flight)

template <int C>
__global__ void __launch_bounds__(kThreads, C <= 64 ? 4 : 2)
conv_fuse_nhwc_bf16(const Params p)
{
    constexpr int PITCH = C * 2 + 16;                       // bytes per staged row: 16-byte rows of an ldmatrix fall in different banks
    constexpr int NT = C / 8, KS = C / 16;
    constexpr bool kRegB = C <= 64;                         // w_fuse as tensor-core fragments in registers (C <= 64), else in shared memory
    constexpr int STAGE = 2 * kPix * PITCH;                 // a tile's cat rows, then its residual rows
    extern __shared__ __align__(16) unsigned char smem[];
    constexpr int NS = Stages<C>::N;
    // [C][PITCH]: w_fuse, row n = output channel; where it goes to registers, it passes through the last stage, which the
    // pipeline fills only after the first barrier of the tile loop
    unsigned char* wsm = smem + (kRegB ? (NS - 1) * STAGE : NS * STAGE);
    static_assert(!kRegB || C * PITCH <= STAGE, "w_fuse fits a stage");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    constexpr int CH = C / 8;                               // 16-byte pieces per row

    // ---- w_fuse: B fragments of mma.m16n8k16 (k = input channel, n = output channel): b0 = W[8 nt + g][16 ks + 2t, + 1],
    //      b1 = the same row, eight input channels on
    uint32_t bw[kRegB ? KS : 1][kRegB ? NT : 1][2];
    for (int e = tid; e < C * CH; e += kThreads) {          // coalesced, 16 bytes per thread
        const int r = e / CH, q = e % CH;
        *reinterpret_cast<uint4*>(wsm + r * PITCH + q * 16) = __ldg(reinterpret_cast<const uint4*>(p.w + (size_t)r * C) + q);
    }
    if (kRegB) {
        __syncthreads();
        const int wmi = lane >> 3, wmr = lane & 7;
        const uint32_t w_lane = tma::smem_u32(wsm) + (uint32_t)(((wmi >> 1) * 8 + wmr) * PITCH + (wmi & 1) * 16);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int n2 = 0; n2 < NT / 2; ++n2) {
                uint32_t b[4];                              // output channels 16 n2 .. + 7 (k halves), then + 8 .. + 15
                tma::toep::ldsm_x4(w_lane + (uint32_t)(n2 * 16 * PITCH) + ks * 32, b);
                bw[kRegB ? ks : 0][kRegB ? 2 * n2 : 0][0] = b[0]; bw[kRegB ? ks : 0][kRegB ? 2 * n2 : 0][1] = b[1];
                bw[kRegB ? ks : 0][kRegB ? 2 * n2 + 1 : 0][0] = b[2]; bw[kRegB ? ks : 0][kRegB ? 2 * n2 + 1 : 0][1] = b[3];
            }
    }
    float bs[NT][2];                                        // this lane's output channels 8n + 2t, + 1
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        bs[n][0] = p.bias ? __bfloat162float(p.bias[8 * n + 2 * t]) : 0.f;
        bs[n][1] = p.bias ? __bfloat162float(p.bias[8 * n + 2 * t + 1]) : 0.f;
    }
    // the weights do not depend on the kernel before this one; the attention channels do
    pdl_wait_primary();

    // a tile's 64 pixels: channels below Ca from `att`, the rest from `idt`, and the residual, 16 bytes per copy
    const long long ntiles = (p.pixels + kPix - 1) / kPix;
    auto stage = [&](long long tile, int buf) {
        const uint32_t xs = tma::smem_u32(smem + buf * STAGE), rs = xs + kPix * PITCH;
        const long long px0 = tile * kPix;
#pragma unroll
        for (int u = 0; u < kPix * CH / kThreads; ++u) {
            const int e = tid + u * kThreads, r = e / CH, q = e % CH;
            const long long px = px0 + r;
            const bool ok = px < p.pixels;
            const size_t at = (size_t)(ok ? px : 0) * C;
            cp_async16(xs + r * PITCH + q * 16, reinterpret_cast<const uint4*>((q * 8 < p.Ca ? p.att : p.idt) + at) + q, ok);
            if (p.residual) cp_async16(rs + r * PITCH + q * 16, reinterpret_cast<const uint4*>(p.residual + at) + q, ok);
        }
        cp_async_commit();
    };
    static_assert(kPix * CH % kThreads == 0, "pieces per thread");

    long long tile = blockIdx.x;
    int buf = 0;
    // one group per tile, empty where there is no tile, so that "all but the NS - 2 newest groups" is always this tile
#pragma unroll
    for (int j = 0; j < NS - 1; ++j) {
        if (tile + j * (long long)gridDim.x < ntiles) stage(tile + j * (long long)gridDim.x, j);
        else cp_async_commit();
    }
    for (; tile < ntiles; tile += gridDim.x, buf = buf + 1 == NS ? 0 : buf + 1) {
        const long long px0 = tile * kPix;
        unsigned char* xsm = smem + buf * STAGE;            // cat of the tile's pixels; later the results
        unsigned char* rsm = xsm + kPix * PITCH;            // the residual of the same pixels
        cp_async_wait<NS - 2>();
        __syncthreads();                                    // the tile is there for everybody; everybody is done with the tile before
        {
            const long long nx = tile + (NS - 1) * (long long)gridDim.x;       // into the buffer of the tile before this one
            if (nx < ntiles) stage(nx, buf == 0 ? NS - 1 : buf - 1);
            else cp_async_commit();
        }

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
            tma::toep::ldsm_x4(a_lane + ks * 32, a);        // rows 0-7 / 8-15 of the warp's pixels, k halves 0 / 1
            if (kRegB) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
                    tma::toep::mma_bf16(acc[nt], a[0], a[1], a[2], a[3], bw[kRegB ? ks : 0][kRegB ? nt : 0][0], bw[kRegB ? ks : 0][kRegB ? nt : 0][1]);
            } else {
#pragma unroll
                for (int n2 = 0; n2 < NT / 2; ++n2) {
                    uint32_t b[4];                          // output channels 16 n2 .. + 7 (k halves), then + 8 .. + 15
                    tma::toep::ldsm_x4(b_lane + (uint32_t)(n2 * 16 * PITCH) + ks * 32, b);
                    tma::toep::mma_bf16(acc[2 * n2], a[0], a[1], a[2], a[3], b[0], b[1]);
                    tma::toep::mma_bf16(acc[2 * n2 + 1], a[0], a[1], a[2], a[3], b[2], b[3]);
                }
            }
        }
        __syncwarp();                                       // a warp's 16 staged pixels are read by that warp alone

        // ---- bias and residual are added in fp32; one rounding to bf16; results staged over the warp's own pixels ----
        // acc[n]: [0], [1] = pixel g, output channels 8n + 2t, + 1; [2], [3] = pixel g + 8
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            const int oc = 8 * n + 2 * t;
            const float b0 = bs[n][0], b1 = bs[n][1];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = warp * 16 + g + 8 * h;
                float v0 = acc[n][2 * h] + b0, v1 = acc[n][2 * h + 1] + b1;
                if (p.residual) {
                    const uint32_t rr = *reinterpret_cast<const uint32_t*>(rsm + r * PITCH + oc * 2);
                    v0 += __uint_as_float(rr << 16);
                    v1 += __uint_as_float(rr & 0xffff0000u);
                }
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
                *reinterpret_cast<uint32_t*>(xsm + r * PITCH + oc * 2) = *reinterpret_cast<const uint32_t*>(&h2);
            }
        }
        __syncwarp();
        // the warp's 16 pixels are 32 C contiguous bytes of the output
#pragma unroll
        for (int u = 0; u < 16 * CH / 32; ++u) {
            const int e = lane + u * 32, r = warp * 16 + e / CH, q = e % CH;
            const long long px = px0 + r;
            if (px < p.pixels)
                *(reinterpret_cast<uint4*>(p.out + (size_t)px * C) + q) = *reinterpret_cast<const uint4*>(xsm + r * PITCH + q * 16);
        }
    }
}

// ---- NCHW bf16, C in {32, 48, 64}: the same product with the roles of the operands exchanged ---------------------------
//   out[n][px] = b[n] + sum_k W[n][k] cat[k][px] (+ residual[n][px]):  D (16 output channels x 8 pixels) = A (W, 16 x 16) x
//   B (16 channels x 8 pixels).  A tile is C channel rows of 128 pixels (256 contiguous bytes each; rows k < Ca from `att`,
//   the rest from `idt`) and the residual's rows, staged with 16-byte asynchronous copies three tiles deep; B comes from the
//   tile by ldmatrix.trans (row pitch 272 bytes: conflict-free), W sits in registers as A fragments; a warp owns 16 pixels
//   and all C output channels, adds bias and residual in fp32, rounds once and writes the results over the residual's tile,
//   from where the block stores whole 256-byte rows.
namespace nchw {
constexpr int kPixN = 128, kThreadsN = 256, kPitchN = kPixN * 2 + 16;
struct Params {
    const __nv_bfloat16* att;         // [B][C][HW]: planes 0 .. Ca-1 are F_res
    const __nv_bfloat16* idt;         // [B][C][HW]: planes Ca .. C-1 are F_idt
    const __nv_bfloat16* w;           // [C][C], row = output channel
    const __nv_bfloat16* bias;        // [C] or nullptr
    const __nv_bfloat16* residual;    // [B][C][HW] or nullptr
    __nv_bfloat16* out;               // [B][C][HW]
    long long HW;                     // a multiple of 8
    int B, C, Ca;
};

template <int C>
__global__ void __launch_bounds__(kThreadsN, 2)
conv_fuse_nchw_bf16(const Params p)
{
    constexpr int MT = C / 16, KS = C / 16, STAGE = 2 * C * kPitchN, NS = 3, WP = C * 2 + 16;
    extern __shared__ __align__(16) unsigned char smem[];
    unsigned char* wsm = smem + (NS - 1) * STAGE;            // w_fuse passes through the last stage on its way to registers
    static_assert(C * WP <= STAGE, "w_fuse fits a stage");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int mi = lane >> 3, mr = lane & 7;
    for (int e = tid; e < C * (C / 8); e += kThreadsN) {
        const int r = e / (C / 8), q = e % (C / 8);
        *reinterpret_cast<uint4*>(wsm + r * WP + q * 16) = __ldg(reinterpret_cast<const uint4*>(p.w + (size_t)r * C) + q);
    }
    __syncthreads();
    uint32_t aw[MT][KS][4];                                  // A fragments: rows 16 mt + (0-7 | 8-15), columns 16 ks + (0-7 | 8-15)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
            tma::toep::ldsm_x4(tma::smem_u32(wsm) + (uint32_t)((16 * mt + (mi & 1) * 8 + mr) * WP + (16 * ks + (mi >> 1) * 8) * 2), aw[mt][ks]);
    float bs[MT][2];                                         // bias of this lane's output channels 16 mt + g, + 8
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        bs[mt][0] = p.bias ? __bfloat162float(p.bias[16 * mt + g]) : 0.f;
        bs[mt][1] = p.bias ? __bfloat162float(p.bias[16 * mt + g + 8]) : 0.f;
    }
    pdl_wait_primary();                                      // the attention planes come from the kernel before this one

    const long long tiles_per_img = (p.HW + kPixN - 1) / kPixN, ntiles = tiles_per_img * p.B;
    auto stage = [&](long long tile, int buf) {
        const long long b = tile / tiles_per_img, p0 = (tile - b * tiles_per_img) * kPixN;
        const uint32_t xs = tma::smem_u32(smem + buf * STAGE), rs = xs + C * kPitchN;
        const size_t img = (size_t)b * C * p.HW;
#pragma unroll
        for (int u = 0; u < C * (kPixN / 8) / kThreadsN; ++u) {
            const int e = tid + u * kThreadsN, ch = e / (kPixN / 8), q = e % (kPixN / 8);
            const bool ok = p0 + q * 8 < p.HW;
            const size_t at = img + (size_t)ch * p.HW + (ok ? p0 + q * 8 : 0);
            cp_async16(xs + ch * kPitchN + q * 16, (ch < p.Ca ? p.att : p.idt) + at, ok);
            if (p.residual) cp_async16(rs + ch * kPitchN + q * 16, p.residual + at, ok);
        }
        cp_async_commit();
    };
    static_assert(C * (kPixN / 8) % kThreadsN == 0, "pieces per thread");
    long long tile = blockIdx.x;
    int buf = 0;
#pragma unroll
    for (int j = 0; j < NS - 1; ++j) {
        if (tile + j * (long long)gridDim.x < ntiles) stage(tile + j * (long long)gridDim.x, j);
        else cp_async_commit();
    }
    for (; tile < ntiles; tile += gridDim.x, buf = buf + 1 == NS ? 0 : buf + 1) {
        const long long b = tile / tiles_per_img, p0 = (tile - b * tiles_per_img) * kPixN;
        unsigned char* xsm = smem + buf * STAGE;
        unsigned char* rsm = xsm + C * kPitchN;
        cp_async_wait<NS - 2>();
        __syncthreads();                                     // the tile is there for everybody; everybody is done with the tile before
        {
            const long long nx = tile + (NS - 1) * (long long)gridDim.x;
            if (nx < ntiles) stage(nx, buf == 0 ? NS - 1 : buf - 1);
            else cp_async_commit();
        }
        float acc[MT][2][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[mt][nt][v] = 0.f;
        const uint32_t b_lane = tma::smem_u32(xsm) + (uint32_t)(((mi & 1) * 8 + mr) * kPitchN + (warp * 16 + (mi >> 1) * 8) * 2);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t bfrag[4];                               // (channels 16 ks .. + 7 | + 8 .. + 15) x (pixels 0-7 | 8-15 of the warp's 16)
            tma::toepn::ldsm_x4_trans(b_lane + (uint32_t)(16 * ks * kPitchN), bfrag);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                tma::toep::mma_bf16(acc[mt][0], aw[mt][ks][0], aw[mt][ks][1], aw[mt][ks][2], aw[mt][ks][3], bfrag[0], bfrag[1]);
                tma::toep::mma_bf16(acc[mt][1], aw[mt][ks][0], aw[mt][ks][1], aw[mt][ks][2], aw[mt][ks][3], bfrag[2], bfrag[3]);
            }
        }
        // acc[mt][nt]: [0], [1] = channel 16 mt + g, pixels 8 nt + 2t, + 1 of the warp's 16; [2], [3] = channel + 8
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t* cell = reinterpret_cast<uint32_t*>(rsm + (16 * mt + g + 8 * h) * kPitchN + (warp * 16 + 8 * nt + 2 * t) * 2);
                    float v0 = acc[mt][nt][2 * h] + bs[mt][h], v1 = acc[mt][nt][2 * h + 1] + bs[mt][h];
                    if (p.residual) {
                        const uint32_t rr = *cell;
                        v0 += __uint_as_float(rr << 16);
                        v1 += __uint_as_float(rr & 0xffff0000u);
                    }
                    const __nv_bfloat162 h2 = __floats2bfloat162_rn(v0, v1);
                    *cell = *reinterpret_cast<const uint32_t*>(&h2);
                }
        __syncthreads();                                     // whole rows are complete
        const size_t img = (size_t)b * C * p.HW;
#pragma unroll
        for (int u = 0; u < C * (kPixN / 8) / kThreadsN; ++u) {
            const int e = tid + u * kThreadsN, ch = e / (kPixN / 8), q = e % (kPixN / 8);
            if (p0 + q * 8 < p.HW)
                *reinterpret_cast<uint4*>(p.out + img + (size_t)ch * p.HW + p0 + q * 8) = *reinterpret_cast<const uint4*>(rsm + ch * kPitchN + q * 16);
        }
    }
}

inline bool applies(int C, int Ca, long long HW, int dtype, int layout, const void* x, const void* out, const void* residual, const void* w) {
    auto al = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; };
    return dtype == 1 /*bf16*/ && layout == kNCHW && (C == 32 || C == 48 || C == 64) && Ca <= C && HW % 8 == 0 && al(x) && al(out) &&
           al(residual) && al(w);
}

// `early`: the kernel may start, and read w, while the kernel before it in the stream still runs (w must then be older than that kernel)
template <int C>
inline cudaError_t launch_c(const Params& p, cudaStream_t st, bool early) {
    const size_t smem = (size_t)3 * 2 * C * kPitchN;
    static bool attr_set[tma::kMaxDevices] = {};
    const int dev = tma::current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(conv_fuse_nchw_bf16<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const long long ntiles = ((p.HW + kPixN - 1) / kPixN) * p.B, cap = 2LL * (tma::sm_count() > 0 ? tma::sm_count() : 148);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(ntiles < cap ? ntiles : cap));
    cfg.blockDim = dim3(kThreadsN);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, conv_fuse_nchw_bf16<C>, p);
}
inline cudaError_t launch(const Params& p, cudaStream_t st, bool early = true) {
    switch (p.C) {
        case 32: return launch_c<32>(p, st, early);
        case 48: return launch_c<48>(p, st, early);
        case 64: return launch_c<64>(p, st, early);
        default: return cudaErrorInvalidValue;
    }
}
}  // namespace nchw

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
inline cudaError_t launch_fast_c(const Params& p, cudaStream_t st, bool early) {
    constexpr int PITCH = C * 2 + 16;
    const size_t smem = (size_t)(2 * Stages<C>::N * kPix + (C <= 64 ? 0 : C)) * PITCH;   // stages of (cat, residual); w_fuse where it is not in registers
    static bool attr_set[tma::kMaxDevices] = {};
    const int dev = tma::current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (!attr_set[dev] && smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(conv_fuse_nhwc_bf16<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const long long ntiles = (p.pixels + kPix - 1) / kPix, cap = (C <= 64 ? 4LL : 2LL) * (tma::sm_count() > 0 ? tma::sm_count() : 148);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(ntiles < cap ? ntiles : cap));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];                             // may start (and stage w_fuse) while the stencil kernel drains
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, conv_fuse_nhwc_bf16<C>, p);
}

inline cudaError_t launch_fast(const Params& p, cudaStream_t st, bool early = true) {
    switch (p.C) {
        case 32: return launch_fast_c<32>(p, st, early);
        case 48: return launch_fast_c<48>(p, st, early);
        case 64: return launch_fast_c<64>(p, st, early);
        case 96: return launch_fast_c<96>(p, st, early);
        case 128: return launch_fast_c<128>(p, st, early);
        default: return cudaErrorInvalidValue;
    }
}

}}  // namespace esc::fuse

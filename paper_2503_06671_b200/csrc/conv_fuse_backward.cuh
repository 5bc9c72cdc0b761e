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
#include "stencil_toeplitz.cuh"
#include "conv_fuse.cuh"

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
        {
            // thread = pixel of the pass: one division per pass (NCHW), 16-byte pieces of the pixel's row (NHWC; the
            // pieces of a row come from the same lines, so all but the first are L1 hits), conflict-free stores
            const long long px = px0 + tid;
            const bool valid = px < pixels;
            if (LAYOUT == kNCHW) {
                const long long b = valid ? px / HW : 0, r = valid ? px - b * HW : 0;
                const size_t base = (size_t)b * C * HW + r;
#pragma unroll 8
                for (int c = 0; c < C; ++c) {
                    float a = 0.f, v = 0.f;
                    if (valid) { a = Elem<T>::to_f32(go[base + (size_t)c * HW]); v = Elem<T>::to_f32(cat[base + (size_t)c * HW]); }
                    gs[c * kPitch + tid] = a;
                    xs[c * kPitch + tid] = v;
                }
            } else {
                constexpr int V = Elem<T>::kVec;
                const size_t base = (size_t)px * C;
#pragma unroll 2
                for (int c0 = 0; c0 < C; c0 += V) {
                    float a[V], v[V];
                    if (valid) {
                        unpack16<T>(*reinterpret_cast<const uint4*>(go + base + c0), a);
                        unpack16<T>(*reinterpret_cast<const uint4*>(cat + base + c0), v);
                    } else {
#pragma unroll
                        for (int i = 0; i < V; ++i) a[i] = v[i] = 0.f;
                    }
#pragma unroll
                    for (int i = 0; i < V; ++i) {
                        gs[(c0 + i) * kPitch + tid] = a[i];
                        xs[(c0 + i) * kPitch + tid] = v[i];
                    }
                }
            }
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

// ---- the same sums on the tensor cores: bf16 NHWC tensors ------------------------------------------------------------
// g_W = go^T [C x pixels] . cat [pixels x C]: one matrix product with the pixels as the contraction axis; bf16 products
// are exact in fp32 and the accumulation is fp32.  A block takes the same runs of pixels as above, 128 at a time (two
// buffers filled with cp.async; pixel rows 16 bytes longer than C channels, so that the eight rows of an ldmatrix fall
// into different banks); warp w owns pixels 16 w .. 16 w + 15 of every piece and the whole C x C accumulator
// (C = 64: 128 registers): per piece C/16 ldmatrix.x4.trans for go (A: channel x pixel out of pixel-major rows), C/16
// for cat (B) and (C/16) x (C/8) mma.sync.m16n8k16, plus C/16 with a B operand of ones for g_b.  At the end the warps
// put their accumulators side by side into shared memory and the block adds them per element in warp order.
namespace mma {
using tma::toep::ldsm_x4_trans; using tma::toep::mma_bf16;
constexpr int kPiece = 128;                                        // pixels per buffer: 16 per warp

template <int C> struct MGeom {
    static constexpr int PITCH = C * 2 + 16;                       // bytes per staged pixel row
    static constexpr int TILE = kPiece * PITCH;                    // one tensor, one buffer
    static constexpr size_t kStageBytes = (size_t)4 * TILE;        // (go, cat) x two buffers
    static constexpr size_t kSumBytes = (size_t)(kThreads / 32) * (C * C + C) * sizeof(float);   // every warp's sums side by side
    static constexpr size_t kSmemBytes = kStageBytes > kSumBytes ? kStageBytes : kSumBytes;
};

template <int C>
__global__ void __launch_bounds__(kThreads, 1)
wgrad_bf16_nhwc(const __nv_bfloat16* __restrict__ cat, const __nv_bfloat16* __restrict__ go, long long pixels, int passes,
                float* __restrict__ part)                          // [gridDim.x][C * C + C]
{
    using G = MGeom<C>;
    constexpr int MT = C / 16, NT = C / 8, CH = C / 8;              // m tiles, n tiles, 16-byte pieces per pixel row
    extern __shared__ __align__(128) unsigned char smb[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mi = lane >> 3, mr = lane & 7;
    // ldmatrix lane address inside a tile: pixel 16 warp + 8 (mi >> 1) + mr, channel half mi & 1 of a 16-channel group
    const uint32_t lane_off = (uint32_t)((16 * warp + 8 * (mi >> 1) + mr) * G::PITCH + (mi & 1) * 16);
    const uint32_t sm0 = tma::smem_u32(smb);
    float acc[MT][NT][4], accb[MT][4];
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[m][n][v] = 0.f;
#pragma unroll
        for (int v = 0; v < 4; ++v) accb[m][v] = 0.f;
    }
    const long long first = (long long)blockIdx.x * passes * kThreads;             // the block's run of pixels
    const long long last = first + (long long)passes * kThreads < pixels ? first + (long long)passes * kThreads : pixels;
    const int pieces = first < last ? (int)((last - first + kPiece - 1) / kPiece) : 0;
    auto stage = [&](int s) {
        const long long p0 = first + (long long)s * kPiece;
        const uint32_t gbuf = sm0 + (uint32_t)((s & 1) * 2 * G::TILE), cbuf = gbuf + G::TILE;
        for (int e = tid; e < kPiece * CH; e += kThreads) {
            const int r = e / CH, q = e % CH;
            const long long px = p0 + r;
            const bool valid = px < last;
            const size_t src = (size_t)(valid ? px : first) * C + q * 8;
            fuse::cp_async16(gbuf + (uint32_t)(r * G::PITCH + q * 16), go + src, valid);
            fuse::cp_async16(cbuf + (uint32_t)(r * G::PITCH + q * 16), cat + src, valid);
        }
        fuse::cp_async_commit();
    };
    if (pieces > 0) stage(0);
    for (int s = 0; s < pieces; ++s) {
        if (s + 1 < pieces) stage(s + 1);
        else fuse::cp_async_commit();
        fuse::cp_async_wait<1>();
        __syncthreads();                                          // piece s is there for every warp
        const uint32_t gbuf = sm0 + (uint32_t)((s & 1) * 2 * G::TILE) + lane_off, cbuf = gbuf + G::TILE;
        uint32_t a[MT][4];
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            ldsm_x4_trans(gbuf + (uint32_t)(m * 32), a[m]);       // go: (channels 0-7 | 8-15 of group m) x (pixels 0-7 | 8-15)
            mma_bf16(accb[m], a[m][0], a[m][1], a[m][2], a[m][3], 0x3F803F80u, 0x3F803F80u);   // times ones: the sum over pixels
        }
#pragma unroll
        for (int n2 = 0; n2 < MT; ++n2) {
            uint32_t b[4];                                        // cat, same arrangement: channel group n2
            ldsm_x4_trans(cbuf + (uint32_t)(n2 * 32), b);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                mma_bf16(acc[m][2 * n2], a[m][0], a[m][1], a[m][2], a[m][3], b[0], b[2]);
                mma_bf16(acc[m][2 * n2 + 1], a[m][0], a[m][1], a[m][2], a[m][3], b[1], b[3]);
            }
        }
        __syncthreads();                                          // the buffer may be refilled
    }
    fuse::cp_async_wait<0>();
    __syncthreads();
    // acc[m][n]: [0], [1] = go channel 16 m + g, cat channels 8 n + 2t, + 1; [2], [3] = go channel + 8.
    // Every warp puts its sums into a region of its own; then they are added per element in warp order.
    constexpr int kPart = C * C + C;
    float* sum = reinterpret_cast<float*>(smb) + warp * kPart;
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int v = 0; v < 4; v += 2)
                *reinterpret_cast<float2*>(sum + (16 * m + g + 8 * (v >> 1)) * C + 8 * n + 2 * t) = make_float2(acc[m][n][v], acc[m][n][v + 1]);
        if (t == 0) {                                             // every column of accb holds the same sum: take column 0
            sum[C * C + 16 * m + g] = accb[m][0];
            sum[C * C + 16 * m + g + 8] = accb[m][2];
        }
    }
    __syncthreads();
    const float* all = reinterpret_cast<const float*>(smb);
    float* out = part + (size_t)blockIdx.x * kPart;
    for (int e = tid; e < kPart; e += kThreads) {
        float v = all[e];
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) v += all[w * kPart + e];
        out[e] = v;
    }
}

// The same for bf16 NCHW tensors (H W a multiple of 8, so that eight consecutive pixels of the flattened list lie in one
// image): rows of a staged tile are channels, 128 pixels long plus 16 bytes; both operands are then the instruction's
// native arrangement (A row-major channel x pixel, B pixel-contiguous per channel): ldmatrix without transposition.
template <int C> struct NGeom {
    static constexpr int PITCH = kPiece * 2 + 16;                  // bytes per staged channel row
    static constexpr int TILE = C * PITCH;
    static constexpr size_t kStageBytes = (size_t)4 * TILE;
    static constexpr size_t kSmemBytes = kStageBytes > MGeom<C>::kSumBytes ? kStageBytes : MGeom<C>::kSumBytes;
};

template <int C>
__global__ void __launch_bounds__(kThreads, 1)
wgrad_bf16_nchw(const __nv_bfloat16* __restrict__ cat, const __nv_bfloat16* __restrict__ go, long long HW, long long pixels,
                int passes, float* __restrict__ part)              // [gridDim.x][C * C + C]
{
    using G = NGeom<C>;
    constexpr int MT = C / 16, NT = C / 8;
    extern __shared__ __align__(128) unsigned char smb[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mi = lane >> 3, mr = lane & 7;
    // ldmatrix lane address inside a tile: channel 8 (mi & 1) + mr of a 16-channel group, pixels 16 warp + 8 (mi >> 1) ..
    const uint32_t lane_off = (uint32_t)((8 * (mi & 1) + mr) * G::PITCH + (16 * warp + 8 * (mi >> 1)) * 2);
    const uint32_t sm0 = tma::smem_u32(smb);
    float acc[MT][NT][4], accb[MT][4];
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[m][n][v] = 0.f;
#pragma unroll
        for (int v = 0; v < 4; ++v) accb[m][v] = 0.f;
    }
    const long long first = (long long)blockIdx.x * passes * kThreads;
    const long long last = first + (long long)passes * kThreads < pixels ? first + (long long)passes * kThreads : pixels;
    const int pieces = first < last ? (int)((last - first + kPiece - 1) / kPiece) : 0;
    auto stage = [&](int s) {
        const long long p0 = first + (long long)s * kPiece;
        const uint32_t gbuf = sm0 + (uint32_t)((s & 1) * 2 * G::TILE), cbuf = gbuf + G::TILE;
        for (int e = tid; e < C * (kPiece / 8); e += kThreads) {
            const int c = e / (kPiece / 8), q = e % (kPiece / 8);
            const long long px = p0 + q * 8;
            const bool valid = px < last;                          // pieces of eight pixels never straddle `last` or an image
            const long long b = valid ? px / HW : 0, r = valid ? px - b * HW : 0;
            const size_t src = ((size_t)b * C + c) * HW + r;
            fuse::cp_async16(gbuf + (uint32_t)(c * G::PITCH + q * 16), go + src, valid);
            fuse::cp_async16(cbuf + (uint32_t)(c * G::PITCH + q * 16), cat + src, valid);
        }
        fuse::cp_async_commit();
    };
    if (pieces > 0) stage(0);
    for (int s = 0; s < pieces; ++s) {
        if (s + 1 < pieces) stage(s + 1);
        else fuse::cp_async_commit();
        fuse::cp_async_wait<1>();
        __syncthreads();
        const uint32_t gbuf = sm0 + (uint32_t)((s & 1) * 2 * G::TILE) + lane_off, cbuf = gbuf + G::TILE;
        uint32_t a[MT][4];
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            tma::toep::ldsm_x4(gbuf + (uint32_t)(m * 16 * G::PITCH), a[m]);   // go: (channels 0-7 | 8-15 of group m) x (pixels 0-7 | 8-15)
            mma_bf16(accb[m], a[m][0], a[m][1], a[m][2], a[m][3], 0x3F803F80u, 0x3F803F80u);
        }
#pragma unroll
        for (int n2 = 0; n2 < MT; ++n2) {
            uint32_t b[4];
            tma::toep::ldsm_x4(cbuf + (uint32_t)(n2 * 16 * G::PITCH), b);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                mma_bf16(acc[m][2 * n2], a[m][0], a[m][1], a[m][2], a[m][3], b[0], b[2]);
                mma_bf16(acc[m][2 * n2 + 1], a[m][0], a[m][1], a[m][2], a[m][3], b[1], b[3]);
            }
        }
        __syncthreads();
    }
    fuse::cp_async_wait<0>();
    __syncthreads();
    constexpr int kPart = C * C + C;
    float* sum = reinterpret_cast<float*>(smb) + warp * kPart;
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int v = 0; v < 4; v += 2)
                *reinterpret_cast<float2*>(sum + (16 * m + g + 8 * (v >> 1)) * C + 8 * n + 2 * t) = make_float2(acc[m][n][v], acc[m][n][v + 1]);
        if (t == 0) {
            sum[C * C + 16 * m + g] = accb[m][0];
            sum[C * C + 16 * m + g + 8] = accb[m][2];
        }
    }
    __syncthreads();
    const float* all = reinterpret_cast<const float*>(smb);
    float* out = part + (size_t)blockIdx.x * kPart;
    for (int e = tid; e < kPart; e += kThreads) {
        float v = all[e];
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) v += all[w * kPart + e];
        out[e] = v;
    }
}
}  // namespace mma

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

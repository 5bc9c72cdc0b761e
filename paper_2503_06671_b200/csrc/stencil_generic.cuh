// Guarded generic stencil for any odd K <= 17, any shape, either layout or element type
// (ESC paper, Section 3.3, Eq. 4 lines 3-4).  One thread per output value: a (TY+K-1) x (TX+K-1)
// halo tile of one channel is staged in shared memory as fp32 with zeros outside the image, the
// per-image merged kernel ZP(dk) + LK^s (Eq. 5) sits beside it, and each thread accumulates its
// K*K taps in fp32.  This is the fall-back when the register-tiled TMA kernel does not apply; it
// is correct everywhere but makes no attempt to be fast.
#pragma once
#include "common.cuh"

namespace esc {

constexpr int kGenTX = 32, kGenTY = 8, kGenMaxK = 17;

// One staged input value of attention channel c: the feature itself, or -- in the decomposed form of
// Eq. 5, (F_att * LK^c) * (ZP(DK) + LK^s) -- the point-wise mix sum_k w_point[c][k] * x[k] of the
// pixel's C_a attention channels (fp32, channel order).  Outside the image both are zero.
template <typename T, int LAYOUT>
__device__ __forceinline__ float staged_value(const T* __restrict__ x, const T* __restrict__ w_point, int b, int c,
                                              int y, int xx, int C, int Ca, int H, int W) {
    if (y < 0 || y >= H || xx < 0 || xx >= W) return 0.f;
    if (w_point == nullptr) return Elem<T>::to_f32(x[elem_index<LAYOUT>(b, c, y, xx, C, H, W)]);
    float v = 0.f;
    for (int k = 0; k < Ca; ++k)
        v = fmaf(Elem<T>::to_f32(w_point[(size_t)c * Ca + k]), Elem<T>::to_f32(x[elem_index<LAYOUT>(b, k, y, xx, C, H, W)]), v);
    return v;
}

// The identity channels (Concat of Eq. 4 line 4) as a strided 2-D copy -- `rows` rows of `row_units` units of
// `unit_bytes` bytes, `stride_units` apart, starting `offset_units` into both tensors -- done by the last
// `blocks` blocks (from `first_block` on) of the same launch that computes the attention channels, so that
// the copy, bound by HBM, runs beside the tail of the arithmetic instead of in a launch of its own after it
// (measured: better than putting the copy blocks first).  blocks == 0: nothing to copy.
struct CopyJob {
    const void* src;
    void* dst;
    long long rows, row_units, stride_units, offset_units;
    int unit_bytes;
    unsigned first_block, blocks;
};

template <typename U>
__device__ __forceinline__ void copy_job_units(const CopyJob& j, unsigned rank, unsigned tid, unsigned nthreads) {
    const U* __restrict__ src = static_cast<const U*>(j.src);
    U* __restrict__ dst = static_cast<U*>(j.dst);
    const long long total = j.rows * j.row_units, step = (long long)j.blocks * nthreads;
    for (long long i = (long long)rank * nthreads + tid; i < total; i += step) {
        const long long r = i / j.row_units, q = i - r * j.row_units;
        const long long e = r * j.stride_units + j.offset_units + q;
        dst[e] = src[e];
    }
}
__device__ __forceinline__ void run_copy_job(const CopyJob& j, unsigned rank, unsigned tid, unsigned nthreads) {
    if (j.unit_bytes == 16) copy_job_units<uint4>(j, rank, tid, nthreads);
    else if (j.unit_bytes == 4) copy_job_units<uint32_t>(j, rank, tid, nthreads);
    else copy_job_units<uint16_t>(j, rank, tid, nthreads);
}

template <typename T, int LAYOUT>
__global__ void __launch_bounds__(kGenTX * kGenTY)
stencil_generic(const T* __restrict__ x, T* __restrict__ out, int C, int Ca, int H, int W, int K,
                const T* __restrict__ w_large, const T* __restrict__ w_point, const float* __restrict__ dk,
                int tiles_x, int tiles_y, const CopyJob job, const float* __restrict__ bias)
{
    __shared__ float tile[(kGenTY + kGenMaxK - 1) * (kGenTX + kGenMaxK - 1)];
    __shared__ float wm[kGenMaxK * kGenMaxK];
    if (job.blocks != 0 && blockIdx.x >= job.first_block) {
        run_copy_job(job, blockIdx.x - job.first_block, threadIdx.y * kGenTX + threadIdx.x, kGenTX * kGenTY);
        return;
    }

    long long bid = blockIdx.x;
    const int tx = (int)(bid % tiles_x); bid /= tiles_x;
    const int ty = (int)(bid % tiles_y); bid /= tiles_y;
    const int c = (int)(bid % Ca);
    const int b = (int)(bid / Ca);
    const int P = (K - 1) / 2;
    const int tid = threadIdx.y * kGenTX + threadIdx.x;
    const int TWp = kGenTX + K - 1, THp = kGenTY + K - 1;
    const int y0 = ty * kGenTY - P, x0 = tx * kGenTX - P;

    pdl_wait_primary();   // dk comes from the preceding kernel when launched as its dependent

    for (int t = tid; t < K * K; t += kGenTX * kGenTY) {
        const int i = t / K, j = t % K;
        float w = Elem<T>::to_f32(w_large[(size_t)c * K * K + t]);
        const int di = i - (P - 1), dj = j - (P - 1);
        if (di >= 0 && di < 3 && dj >= 0 && dj < 3) w += dk[((size_t)b * Ca + c) * 9 + di * 3 + dj];
        wm[t] = w;
    }
    for (int t = tid; t < TWp * THp; t += kGenTX * kGenTY) {
        const int r = t / TWp, q = t % TWp;
        tile[t] = staged_value<T, LAYOUT>(x, w_point, b, c, y0 + r, x0 + q, C, Ca, H, W);
    }
    __syncthreads();

    const int oy = ty * kGenTY + threadIdx.y, ox = tx * kGenTX + threadIdx.x;
    if (oy >= H || ox >= W) return;
    float acc = bias ? bias[(size_t)b * Ca + c] : 0.f;   // the backward pass adds a constant per (image, channel)
    for (int i = 0; i < K; ++i) {
        const float* trow = tile + (threadIdx.y + i) * TWp + threadIdx.x;
        const float* wrow = wm + i * K;
        for (int j = 0; j < K; ++j) acc = fmaf(wrow[j], trow[j], acc);
    }
    out[elem_index<LAYOUT>(b, c, oy, ox, C, H, W)] = Elem<T>::from_f32(acc);
}

// Register-tiled variant for K = 13 (the paper's kernel size) on any layout and element type: the
// same staging as above, but a 64 x 64 output tile per block and a 4 x 8 patch of outputs per thread.
// The loop runs over the 16 input rows a patch touches: a row costs five 16-byte reads and is used by
// up to four output rows, each with its kernel row (four broadcast 16-byte reads), 104 FMAs apiece.
// It serves the fp32 and NCHW cases that the TMA kernel does not take.
// Three geometries: 64 x 64 tiles with 4 x 8 patches (most arithmetic per load: large problems), and 64 x 32 tiles with
// 2 x 8 patches or 32 x 32 tiles with 2 x 4 patches for launches that would otherwise leave most SMs with one block of
// four warps or none (a 320x180 fp32 map is 240 of the large tiles: its stencil stage takes 25 us with them, 18 us with
// 480 of the middle ones; a 64x64 map 15 us as 16 large tiles, 6 us as 64 of the smallest).
constexpr int kRtK = 13;
template <int TX_, int TY_, int OX_, int OY_>
struct RtGeom {
    static constexpr int TX = TX_, TY = TY_, OX = OX_, OY = OY_;
    static constexpr int Pitch = TX + kRtK - 1;                 // floats per staged row, a multiple of 4
    static constexpr int Rows = TY + kRtK - 1;
    static constexpr int Threads = (TX / OX) * (TY / OY);       // 128
    static_assert(Pitch % 4 == 0 && OX % 4 == 0 && Threads == 128, "geometry");
};
using RtLarge = RtGeom<64, 64, 8, 4>;
using RtSmall = RtGeom<64, 32, 8, 2>;
using RtTiny = RtGeom<32, 32, 4, 2>;
constexpr int kRtTX = RtLarge::TX, kRtTY = RtLarge::TY, kRtThreads = 128;

template <typename T, int LAYOUT, class G>
__global__ void __launch_bounds__(128)
stencil_k13_regtile(const T* __restrict__ x, T* __restrict__ out, int C, int Ca, int H, int W,
                    const T* __restrict__ w_large, const T* __restrict__ w_point, const float* __restrict__ dk,
                    int tiles_x, int tiles_y, const CopyJob job, const float* __restrict__ bias)
{
    constexpr int kRtTX = G::TX, kRtTY = G::TY, kRtOX = G::OX, kRtOY = G::OY, kRtPitch = G::Pitch, kRtRows = G::Rows, kRtThreads = G::Threads;
    __shared__ __align__(16) float tile[kRtRows * kRtPitch];
    __shared__ __align__(16) float wm[kRtK * 16];      // merged kernel, rows padded to 16 taps
    if (job.blocks != 0 && blockIdx.x >= job.first_block) {
        run_copy_job(job, blockIdx.x - job.first_block, threadIdx.x, kRtThreads);
        return;
    }

    long long bid = blockIdx.x;
    const int tx = (int)(bid % tiles_x); bid /= tiles_x;
    const int ty = (int)(bid % tiles_y); bid /= tiles_y;
    const int c = (int)(bid % Ca);
    const int b = (int)(bid / Ca);
    constexpr int P = (kRtK - 1) / 2;
    const int tid = threadIdx.x;
    const int y0 = ty * kRtTY - P, x0 = tx * kRtTX - P;

    // eight loads of a thread are in flight before the first is stored: the staging is a chain of round trips otherwise
    for (int t0 = tid; t0 < kRtRows * kRtPitch; t0 += 8 * kRtThreads) {
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int t = t0 + u * kRtThreads, r = t / kRtPitch, q = t % kRtPitch;
            v[u] = t < kRtRows * kRtPitch ? staged_value<T, LAYOUT>(x, w_point, b, c, y0 + r, x0 + q, C, Ca, H, W) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int t = t0 + u * kRtThreads;
            if (t < kRtRows * kRtPitch) tile[t] = v[u];
        }
    }
    pdl_wait_primary();   // dk comes from the preceding kernel when launched as its dependent
    for (int t = tid; t < kRtK * 16; t += kRtThreads) {
        const int i = t / 16, j = t % 16;
        float w = 0.f;
        if (j < kRtK) {
            w = Elem<T>::to_f32(w_large[((size_t)c * kRtK + i) * kRtK + j]);
            const int di = i - (P - 1), dj = j - (P - 1);
            if (di >= 0 && di < 3 && dj >= 0 && dj < 3) w += dk[((size_t)b * Ca + c) * 9 + di * 3 + dj];
        }
        wm[t] = w;
    }
    __syncthreads();

    const int lx = tid % (kRtTX / kRtOX), ly = tid / (kRtTX / kRtOX);
    float acc[kRtOY][kRtOX];
    const float acc0 = bias ? bias[(size_t)b * Ca + c] : 0.f;   // the backward pass adds a constant per (image, channel)
#pragma unroll
    for (int a = 0; a < kRtOY; ++a)
#pragma unroll
        for (int o = 0; o < kRtOX; ++o) acc[a][o] = acc0;
#pragma unroll 1
    for (int r = 0; r < kRtOY + kRtK - 1; ++r) {          // input row r of the patch window
        float in[kRtOX + kRtK - 1];
        const float4* trow = reinterpret_cast<const float4*>(tile + (ly * kRtOY + r) * kRtPitch + lx * kRtOX);
#pragma unroll
        for (int v = 0; v < (kRtOX + kRtK - 1) / 4; ++v) {
            const float4 q = trow[v];
            in[4 * v] = q.x; in[4 * v + 1] = q.y; in[4 * v + 2] = q.z; in[4 * v + 3] = q.w;
        }
#pragma unroll
        for (int a = 0; a < kRtOY; ++a) {
            const int i = r - a;                           // kernel row that maps input row r to output row a
            if (i >= 0 && i < kRtK) {
                float w[16];
                const float4* wrow = reinterpret_cast<const float4*>(wm + i * 16);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const float4 q = wrow[v];
                    w[4 * v] = q.x; w[4 * v + 1] = q.y; w[4 * v + 2] = q.z; w[4 * v + 3] = q.w;
                }
#pragma unroll
                for (int j = 0; j < kRtK; ++j)
#pragma unroll
                    for (int o = 0; o < kRtOX; ++o) acc[a][o] = fmaf(w[j], in[o + j], acc[a][o]);
            }
        }
    }
    const int ox0 = tx * kRtTX + lx * kRtOX;
#pragma unroll
    for (int a = 0; a < kRtOY; ++a) {
        const int oy = ty * kRtTY + ly * kRtOY + a;
        if (oy < H) {
#pragma unroll
            for (int o = 0; o < kRtOX; ++o)
                if (ox0 + o < W) out[elem_index<LAYOUT>(b, c, oy, ox0 + o, C, H, W)] = Elem<T>::from_f32(acc[a][o]);
        }
    }
}

// Copy of the channels that the module leaves untouched (Concat of Eq. 4 line 4), written as a
// strided 2-D copy: `rows` rows of `row_units` units, `stride_units` apart, starting
// `offset_units` into both tensors.  U is the widest unit all three quantities divide into.
template <typename U>
__global__ void __launch_bounds__(256)
copy_through(const U* __restrict__ src, U* __restrict__ dst, long long rows, long long row_units,
             long long stride_units, long long offset_units)
{
    const long long total = rows * row_units;
    const long long step = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += step) {
        const long long r = i / row_units, q = i - r * row_units;
        const long long e = r * stride_units + offset_units + q;
        dst[e] = src[e];
    }
}

}  // namespace esc

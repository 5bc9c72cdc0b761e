// Backward pass of the ConvAttn forward (ESC paper, Section 3.3, Eq. 4, depth-wise LK; one-layer estimator, or the
// two-layer estimator of Eq. 4 line 2 at the end of this file), the chain rule written out.  With go = dL/dout and Wm[b,c] = LK[c] + ZP(dk[b,c]):
//
//   g_tap[b,c,i,j] = sum_{y,x} go[b,c,y,x] * x~[b,c,y+i-6,x+j-6]      per-image tap gradient  (kernel tap_grad)
//   g_lk = sum_b g_tap;   g_dk = central 3x3 of g_tap;   g_b = sum_b g_dk;   g_W[o,k] = sum_b g_dk[b,o] g[b,k]
//   g_g[b,k] = sum_o W[o,k] g_dk[b,o]                                                        (kernel finish)
//   g_x[b,c] = go[b,c] (*) flip(Wm[b,c]) + g_g[b,c] / (H W)   (c < C_a),   g_x[b,c] = go[b,c]  (c >= C_a)
//
// The last line is the forward stencil applied to go with both kernels rotated by 180 degrees and a
// per-(image, channel) constant added, so it runs on the forward kernels; `finish` prepares the rotated
// kernels and the constants for it.  Every reduction is done in a fixed order: results are reproducible.
#pragma once
#include "common.cuh"
#include "stencil_generic.cuh"
#include "gap_dynkernel.cuh"

namespace esc { namespace bwd {

constexpr int K = 13, P = 6, TAPS = K * K;
constexpr int TX = 64, TY = 64, OX = 8, OY = 4;           // tile of go per block, patch of go per thread
constexpr int XP = TX + K - 1;                            // 76 floats per staged x row (a multiple of 4)
constexpr int XR = TY + K - 1;                            // 76 staged x rows
constexpr int kThreads = (TX / OX) * (TY / OY);           // 128
constexpr int kSlot = 176;                                // floats per (image, channel, tile): 169 taps, sum of x, padding
static_assert(XP % 4 == 0 && TAPS + 1 <= kSlot, "layout");

// ---- kernel 1: per-tile partial tap gradients and partial sums of x ---------------------------------------
// Block = (image b, attention channel c, 64x64 tile).  The x halo tile (zeros outside the image) and the go
// tile (zeros outside) are staged in shared memory as fp32; a thread keeps its 4x8 patch of go in registers
// and, for every kernel row i, reads the four x rows its patch meets (five 16-byte reads each) and forms the
// 13 partial sums of that row: 416 FMAs per 20 reads.  The 13 sums are then added over the block in a fixed
// order (shuffle butterfly inside a warp, warps in order).
template <typename T, int LAYOUT>
__global__ void __launch_bounds__(kThreads)
tap_grad(const T* __restrict__ x, const T* __restrict__ go, int C, int Ca, int H, int W, int tiles_x, int tiles_y,
         float* __restrict__ part)      // [B][Ca][tiles][kSlot]
{
    __shared__ __align__(16) float xt[XR * XP];
    __shared__ __align__(16) float gt[TY * TX];
    __shared__ float red[kThreads / 32][16];

    long long bid = blockIdx.x;
    const int tiles = tiles_x * tiles_y;
    const int tile = (int)(bid % tiles); bid /= tiles;
    const int c = (int)(bid % Ca);
    const int b = (int)(bid / Ca);
    const int tx = tile % tiles_x, ty = tile / tiles_x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int y0 = ty * TY, x0 = tx * TX;

    for (int t = tid; t < XR * XP; t += kThreads) {
        const int r = t / XP, q = t % XP;
        const int y = y0 - P + r, xx = x0 - P + q;
        xt[t] = (y >= 0 && y < H && xx >= 0 && xx < W) ? Elem<T>::to_f32(x[elem_index<LAYOUT>(b, c, y, xx, C, H, W)]) : 0.f;
    }
    for (int t = tid; t < TY * TX; t += kThreads) {
        const int r = t / TX, q = t % TX;
        const int y = y0 + r, xx = x0 + q;
        gt[t] = (y < H && xx < W) ? Elem<T>::to_f32(go[elem_index<LAYOUT>(b, c, y, xx, C, H, W)]) : 0.f;
    }
    __syncthreads();

    const int lx = tid % (TX / OX), ly = tid / (TX / OX);
    float g[OY][OX];
    float sx = 0.f;                                       // sum of x over the patch (for the GAP of this image)
#pragma unroll
    for (int a = 0; a < OY; ++a) {
        const float4* gr = reinterpret_cast<const float4*>(gt + (ly * OY + a) * TX + lx * OX);
        const float4 q0 = gr[0], q1 = gr[1];
        g[a][0] = q0.x; g[a][1] = q0.y; g[a][2] = q0.z; g[a][3] = q0.w;
        g[a][4] = q1.x; g[a][5] = q1.y; g[a][6] = q1.z; g[a][7] = q1.w;
        const float4* xr = reinterpret_cast<const float4*>(xt + (ly * OY + a + P) * XP + lx * OX + P - 2);   // 16-byte aligned: P - 2 = 4
        // the patch's own pixels sit at columns lx*OX + P .. +7: floats 2..9 of the three reads from column lx*OX + 4
        const float4 u0 = xr[0], u1 = xr[1], u2 = xr[2];
        sx += (u0.z + u0.w) + (u1.x + u1.y + u1.z + u1.w) + (u2.x + u2.y);
    }
    float* slot = part + (((size_t)b * Ca + c) * tiles + tile) * kSlot;

#pragma unroll 1
    for (int i = 0; i < K; ++i) {
        float s[K];
#pragma unroll
        for (int j = 0; j < K; ++j) s[j] = 0.f;
#pragma unroll
        for (int a = 0; a < OY; ++a) {
            float in[OX + K - 1];                         // x row (ly*OY + a + i), columns lx*OX .. lx*OX + 19
            const float4* xr = reinterpret_cast<const float4*>(xt + (ly * OY + a + i) * XP + lx * OX);
#pragma unroll
            for (int v = 0; v < (OX + K - 1) / 4; ++v) {
                const float4 q = xr[v];
                in[4 * v] = q.x; in[4 * v + 1] = q.y; in[4 * v + 2] = q.z; in[4 * v + 3] = q.w;
            }
#pragma unroll
            for (int j = 0; j < K; ++j)
#pragma unroll
                for (int o = 0; o < OX; ++o) s[j] = fmaf(g[a][o], in[o + j], s[j]);
        }
        // block sum of the 13 values, fixed order
#pragma unroll
        for (int j = 0; j < K; ++j)
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) s[j] += __shfl_xor_sync(0xffffffffu, s[j], o);
        if (lane == 0) {
#pragma unroll
            for (int j = 0; j < K; ++j) red[warp][j] = s[j];
        }
        __syncthreads();
        if (tid < K) {
            float t = 0.f;
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) t += red[w][tid];
            slot[i * K + tid] = t;
        }
        __syncthreads();
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, o);
    if (lane == 0) red[warp][0] = sx;
    __syncthreads();
    if (tid == 0) {
        float t = 0.f;
        for (int w = 0; w < kThreads / 32; ++w) t += red[w][0];
        slot[TAPS] = t;
    }
}

// ---- kernel 1, NHWC form: eight channels per block -----------------------------------------------------------
// In NHWC a block per channel would fetch every pixel's line once per channel with 2-byte loads.  Here a block
// takes eight neighbouring channels (16 bytes of a bf16 pixel, 32 of an fp32 one) of a 32x32 tile: pixels are
// read with 16-byte loads and spread over eight planar fp32 tiles in shared memory; warp w then works on channel
// w on its own (8x4 patch of go per lane), so the block sum of the 13 values is one shuffle butterfly.
namespace n8 {
constexpr int TX = 32, TY = 32, CH = 8;
constexpr int XP = TX + K - 1, XR = TY + K - 1;          // 44 x 44 staged x per channel (44 is a multiple of 4)
constexpr int kThreads = CH * 32;                        // 256
constexpr size_t kSmemBytes = (size_t)CH * (XR * XP + TY * TX) * sizeof(float);   // 94,720
static_assert(XP % 4 == 0, "16-byte reads of staged rows");
}  // namespace n8

template <typename T>
__global__ void __launch_bounds__(n8::kThreads)
tap_grad_nhwc8(const T* __restrict__ x, const T* __restrict__ go, int C, int Ca, int H, int W, int tiles_x, int tiles_y,
               float* __restrict__ part)      // [B][Ca][tiles][kSlot]
{
    constexpr int TX = n8::TX, TY = n8::TY, CH = n8::CH, XP = n8::XP, XR = n8::XR, kThreads = n8::kThreads;
    constexpr int V = Elem<T>::kVec;                      // elements per 16-byte load: 8 (bf16) or 4 (fp32)
    extern __shared__ __align__(16) float sm[];
    float* xt = sm;                                       // [CH][XR*XP]
    float* gt = sm + CH * XR * XP;                        // [CH][TY*TX]

    long long bid = blockIdx.x;
    const int tiles = tiles_x * tiles_y, octets = Ca / CH;
    const int tile = (int)(bid % tiles); bid /= tiles;
    const int oct = (int)(bid % octets);
    const int b = (int)(bid / octets);
    const int tx = tile % tiles_x, ty = tile / tiles_x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int y0 = ty * TY, x0 = tx * TX;
    const T* xb = x + (size_t)b * H * W * C + oct * CH;
    const T* gb = go + (size_t)b * H * W * C + oct * CH;

    for (int t = tid; t < XR * XP * (CH / V); t += kThreads) {
        const int h = t % (CH / V), pix = t / (CH / V);   // which 16-byte piece of the pixel's eight channels
        const int r = pix / XP, q = pix % XP;
        const int y = y0 - P + r, xx = x0 - P + q;
        float f[V];
        if (y >= 0 && y < H && xx >= 0 && xx < W)
            unpack16<T>(__ldg(reinterpret_cast<const uint4*>(xb + ((size_t)y * W + xx) * C + h * V)), f);
        else {
#pragma unroll
            for (int v = 0; v < V; ++v) f[v] = 0.f;
        }
#pragma unroll
        for (int v = 0; v < V; ++v) xt[(h * V + v) * (XR * XP) + pix] = f[v];
    }
    for (int t = tid; t < TY * TX * (CH / V); t += kThreads) {
        const int h = t % (CH / V), pix = t / (CH / V);
        const int r = pix / TX, q = pix % TX;
        const int y = y0 + r, xx = x0 + q;
        float f[V];
        if (y < H && xx < W)
            unpack16<T>(__ldg(reinterpret_cast<const uint4*>(gb + ((size_t)y * W + xx) * C + h * V)), f);
        else {
#pragma unroll
            for (int v = 0; v < V; ++v) f[v] = 0.f;
        }
#pragma unroll
        for (int v = 0; v < V; ++v) gt[(h * V + v) * (TY * TX) + pix] = f[v];
    }
    __syncthreads();

    const float* xc = xt + warp * (XR * XP);              // this warp's channel
    const float* gc = gt + warp * (TY * TX);
    // A lane's patch is 8 rows x 4 columns here: the eight lanes that share a 16-byte read phase then sit
    // side by side (16 bytes apart, 128 contiguous bytes) and the reads are free of bank conflicts.
    constexpr int PY = 8, PX = 4;
    static_assert((TX / PX) * (TY / PY) == 32, "one warp covers a channel's tile");
    const int lx = lane % (TX / PX), ly = lane / (TX / PX);
    float g[PY][PX];
    float sx = 0.f;
#pragma unroll
    for (int a = 0; a < PY; ++a) {
        const float4 q0 = *reinterpret_cast<const float4*>(gc + (ly * PY + a) * TX + lx * PX);
        g[a][0] = q0.x; g[a][1] = q0.y; g[a][2] = q0.z; g[a][3] = q0.w;
        const float4* xr = reinterpret_cast<const float4*>(xc + (ly * PY + a + P) * XP + lx * PX + P - 2);
        const float4 u0 = xr[0], u1 = xr[1];              // the patch's own pixels are floats 2..5 of these
        sx += (u0.z + u0.w) + (u1.x + u1.y);
    }
    float* slot = part + (((size_t)b * Ca + oct * CH + warp) * tiles + tile) * kSlot;

#pragma unroll 1
    for (int i = 0; i < K; ++i) {
        float s[K];
#pragma unroll
        for (int j = 0; j < K; ++j) s[j] = 0.f;
#pragma unroll
        for (int a = 0; a < PY; ++a) {
            float in[PX + K - 1];                         // 16 floats: four 16-byte reads
            const float4* xr = reinterpret_cast<const float4*>(xc + (ly * PY + a + i) * XP + lx * PX);
#pragma unroll
            for (int v = 0; v < (PX + K - 1) / 4; ++v) {
                const float4 q = xr[v];
                in[4 * v] = q.x; in[4 * v + 1] = q.y; in[4 * v + 2] = q.z; in[4 * v + 3] = q.w;
            }
#pragma unroll
            for (int j = 0; j < K; ++j)
#pragma unroll
                for (int o = 0; o < PX; ++o) s[j] = fmaf(g[a][o], in[o + j], s[j]);
        }
#pragma unroll
        for (int j = 0; j < K; ++j)
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) s[j] += __shfl_xor_sync(0xffffffffu, s[j], o);
        // after the butterfly every lane holds all 13 sums: lane j writes the j-th
#pragma unroll
        for (int j = 0; j < K; ++j)
            if (lane == j) slot[i * K + j] = s[j];
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) sx += __shfl_xor_sync(0xffffffffu, sx, o);
    if (lane == 0) slot[TAPS] = sx;
}

// ---- kernel 2a: add the tiles of one (image, channel) in a fixed order -----------------------------------------
// Block = (image, channel); kSumGroups groups of 192 threads take every kSumGroups-th tile each (eight loads in
// flight, added in order), then the groups' sums are added in group order.
constexpr int kSumGroups = 4, kSumThreads = 192 * kSumGroups;
__global__ void __launch_bounds__(kSumThreads)
sum_tiles(const float* __restrict__ part, int tiles, float* __restrict__ gtap)   // gtap [B*Ca][kSlot]
{
    __shared__ float acc[kSumGroups][192];
    const size_t bc = blockIdx.x;
    const int t = threadIdx.x % 192, grp = threadIdx.x / 192;
    if (t <= TAPS) {
        const float* p = part + bc * tiles * kSlot + t;
        float s = 0.f;
#pragma unroll 8
        for (int k = grp; k < tiles; k += kSumGroups) s += p[(size_t)k * kSlot];
        acc[grp][t] = s;
    }
    __syncthreads();
    if (grp == 0 && t <= TAPS) {
        float s = acc[0][t];
#pragma unroll
        for (int q = 1; q < kSumGroups; ++q) s += acc[q][t];
        gtap[bc * kSlot + t] = s;
    }
}

// ---- kernel 2b: everything small; every output element is independent, a few blocks share them ------------
// From g_tap [B][Ca][169 + sum x]: g_lk, g_b, g_W (fp32 outputs), and for the stencil pass that follows the
// kernels rotated by 180 degrees -- w_flip (element type T), dk_flip [B][Ca][9] -- and the constants
// bias[b][c] = g_g[b,c] / (H W).  g[b,k] = sum x / (H W) and dk = b_dyn + W g are recomputed here.
constexpr int kFinishRoles = 6, kFinishBlocks = 32 * kFinishRoles;
template <typename T>
__global__ void __launch_bounds__(256)
finish(const float* __restrict__ gtap, int B, int Ca, int H, int W, int KK, const T* __restrict__ w_large,
       const T* __restrict__ w_dyn, const T* __restrict__ b_dyn, float* __restrict__ g_lk, float* __restrict__ g_w,
       float* __restrict__ g_b, T* __restrict__ w_flip, float* __restrict__ dk_flip, float* __restrict__ bias)
{
    // Six independent jobs; each takes a sixth of the grid, so that their chains of dependent loads run side by side
    // instead of one after the other in every thread.
    const int per_role = gridDim.x / kFinishRoles, role = blockIdx.x / per_role;
    const int tid = (blockIdx.x % per_role) * blockDim.x + threadIdx.x, nth = per_role * blockDim.x;
    const float inv_hw = 1.0f / ((float)H * (float)W);
    auto gdk = [&](int b, int o) {                        // o = c*9 + i*3 + j -> central 3x3 of the tap gradient
        const int c = o / 9, i = (o % 9) / 3, j = o % 3;
        return gtap[((size_t)b * Ca + c) * kSlot + (i + P - 1) * K + (j + P - 1)];
    };
    auto gmean = [&](int b, int k) { return gtap[((size_t)b * Ca + k) * kSlot + TAPS] * inv_hw; };
    // A large kernel of size KK < 13 sits in the middle of the 13 x 13 taps whose gradients gtap holds.
    const int off = (K - KK) / 2, taps = KK * KK;
    if (role == 0 && g_lk)
        for (int e = tid; e < Ca * taps; e += nth) {
            const int c = e / taps, t = (e % taps) / KK + off, u = (e % taps) % KK + off;
            float s = 0.f;
#pragma unroll 8
            for (int b = 0; b < B; ++b) s += gtap[((size_t)b * Ca + c) * kSlot + t * K + u];
            g_lk[e] = s;
        }
    if (role == 1 && g_b)
        for (int o = tid; o < 9 * Ca; o += nth) {
            float s = 0.f;
#pragma unroll 8
            for (int b = 0; b < B; ++b) s += gdk(b, o);
            g_b[o] = s;
        }
    if (role == 2 && g_w)
        for (int e = tid; e < 9 * Ca * Ca; e += nth) {
            const int o = e / Ca, k = e % Ca;
            float s = 0.f;
#pragma unroll 8
            for (int b = 0; b < B; ++b) s = fmaf(gdk(b, o), gmean(b, k), s);
            g_w[e] = s;
        }
    if (role == 3)
    for (int e = tid; e < Ca * taps; e += nth) {
        const int c = e / taps, t = e % taps;
        w_flip[(size_t)c * taps + (taps - 1 - t)] = w_large[e];
    }
    if (role == 4)
    for (int e = tid; e < B * Ca * 9; e += nth) {
        const int b = e / (9 * Ca), o = e % (9 * Ca), c = o / 9, t = o % 9;
        float s = Elem<T>::to_f32(b_dyn[o]);
#pragma unroll 8
        for (int k = 0; k < Ca; ++k) s = fmaf(Elem<T>::to_f32(w_dyn[(size_t)o * Ca + k]), gmean(b, k), s);
        dk_flip[((size_t)b * Ca + c) * 9 + (8 - t)] = s;
    }
    if (role == 5) {
        // bias[b][k] = sum_o W[o][k] g_dk[b][o] / (H W): a warp per element, lane = channel c (nine taps each, all loads
        // independent), then a fixed butterfly over the lanes
        const int lane = threadIdx.x & 31, wid = tid >> 5, nw = nth >> 5;
        for (int e = wid; e < B * Ca; e += nw) {
            const int b = e / Ca, k = e % Ca;
            float s = 0.f;
            for (int c = lane; c < Ca; c += 32) {
                const float* gt = gtap + ((size_t)b * Ca + c) * kSlot + (P - 1) * K + (P - 1);
#pragma unroll
                for (int ij = 0; ij < 9; ++ij)
                    s = fmaf(Elem<T>::to_f32(w_dyn[(size_t)(c * 9 + ij) * Ca + k]), gt[(ij / 3) * K + ij % 3], s);
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0) bias[e] = s * inv_hw;
        }
    }
}

// ---- the estimator as Eq. 4 line 2 writes it: two layers with the exact GELU between them ---------------------
//   t = W_down g + b_down,  a = phi(t),  dk = W_up a + b_up;   phi'(t) = Phi(t) + t n(t)
//   g_a[b,m] = sum_o W_up[o,m] g_dk[b,o],   g_t = g_a * phi'(t),   g_g[b,k] = sum_m W_down[m,k] g_t[b,m]
//   g_b_up = sum_b g_dk,  g_W_up[o,m] = sum_b g_dk[b,o] a[b,m],  g_b_down = sum_b g_t,  g_W_down[m,k] = sum_b g_t[b,m] g[b,k]
__device__ __forceinline__ float gelu_exact_prime(float t) {
    return 0.5f * erfcf(-0.70710678118654752f * t) + t * 0.3989422804014327f * expf(-0.5f * t * t);
}

// kernel 2c: one block per image -- the estimator's forward values and the part of the chain that belongs to one
// image: a and g_t go to the workspace for the sums over images, dk (rotated) and the GAP-path constant to the
// stencil pass that follows.  Dynamic shared memory: (10 Ca + 3 hidden) floats.
template <typename T>
__global__ void __launch_bounds__(256)
mlp_image(const float* __restrict__ gtap, int Ca, int hidden, int H, int W, const T* __restrict__ w_down,
          const T* __restrict__ b_down, const T* __restrict__ w_up, const T* __restrict__ b_up,
          float* __restrict__ act, float* __restrict__ gt, float* __restrict__ dk_flip, float* __restrict__ bias)
{
    extern __shared__ float sm[];
    float* gm = sm;                    // [Ca] pooled means
    float* gd = gm + Ca;               // [9 Ca] g_dk of this image
    float* tt = gd + 9 * Ca;           // [hidden] pre-activations
    float* aa = tt + hidden;           // [hidden] activations
    float* gs = aa + hidden;           // [hidden] g_t
    const int b = blockIdx.x, tid = threadIdx.x, nth = blockDim.x;
    const float inv_hw = 1.0f / ((float)H * (float)W);
    for (int k = tid; k < Ca; k += nth) gm[k] = gtap[((size_t)b * Ca + k) * kSlot + TAPS] * inv_hw;
    for (int o = tid; o < 9 * Ca; o += nth) {
        const int c = o / 9, i = (o % 9) / 3, j = o % 3;
        gd[o] = gtap[((size_t)b * Ca + c) * kSlot + (i + P - 1) * K + (j + P - 1)];
    }
    __syncthreads();
    for (int m = tid; m < hidden; m += nth) {
        float t = Elem<T>::to_f32(b_down[m]);
        for (int k = 0; k < Ca; ++k) t = fmaf(Elem<T>::to_f32(w_down[(size_t)m * Ca + k]), gm[k], t);
        tt[m] = t;
        aa[m] = gelu_exact(t);
        act[(size_t)b * hidden + m] = aa[m];
    }
    __syncthreads();
    for (int o = tid; o < 9 * Ca; o += nth) {
        float s = Elem<T>::to_f32(b_up[o]);
        for (int m = 0; m < hidden; ++m) s = fmaf(Elem<T>::to_f32(w_up[(size_t)o * hidden + m]), aa[m], s);
        dk_flip[(size_t)b * Ca * 9 + (o / 9) * 9 + (8 - o % 9)] = s;
    }
    for (int m = tid; m < hidden; m += nth) {
        float s = 0.f;
        for (int o = 0; o < 9 * Ca; ++o) s = fmaf(Elem<T>::to_f32(w_up[(size_t)o * hidden + m]), gd[o], s);
        s *= gelu_exact_prime(tt[m]);
        gs[m] = s;
        gt[(size_t)b * hidden + m] = s;
    }
    __syncthreads();
    for (int k = tid; k < Ca; k += nth) {
        float s = 0.f;
        for (int m = 0; m < hidden; ++m) s = fmaf(Elem<T>::to_f32(w_down[(size_t)m * Ca + k]), gs[m], s);
        bias[(size_t)b * Ca + k] = s * inv_hw;
    }
}

// kernel 2d: the sums over images (fixed order) and the rotated LK; six jobs on separate blocks.
constexpr int kMlpRoles = 6, kMlpBlocks = 32 * kMlpRoles;
template <typename T>
__global__ void __launch_bounds__(256)
mlp_weights(const float* __restrict__ gtap, const float* __restrict__ act, const float* __restrict__ gt, int B, int Ca,
            int hidden, int H, int W, int KK, const T* __restrict__ w_large, float* __restrict__ g_lk, float* __restrict__ g_wd,
            float* __restrict__ g_bd, float* __restrict__ g_wu, float* __restrict__ g_bu, T* __restrict__ w_flip)
{
    const int per_role = gridDim.x / kMlpRoles, role = blockIdx.x / per_role;
    const int tid = (blockIdx.x % per_role) * blockDim.x + threadIdx.x, nth = per_role * blockDim.x;
    const float inv_hw = 1.0f / ((float)H * (float)W);
    auto gdk = [&](int b, int o) {
        const int c = o / 9, i = (o % 9) / 3, j = o % 3;
        return gtap[((size_t)b * Ca + c) * kSlot + (i + P - 1) * K + (j + P - 1)];
    };
    const int off = (K - KK) / 2, taps = KK * KK;      // a smaller large kernel sits in the middle of the 13 x 13 taps
    if (role == 0 && g_lk)
        for (int e = tid; e < Ca * taps; e += nth) {
            const int c = e / taps, t = (e % taps) / KK + off, u = (e % taps) % KK + off;
            float s = 0.f;
#pragma unroll 8
            for (int b = 0; b < B; ++b) s += gtap[((size_t)b * Ca + c) * kSlot + t * K + u];
            g_lk[e] = s;
        }
    if (role == 1)
        for (int e = tid; e < Ca * taps; e += nth) {
            const int c = e / taps, t = e % taps;
            w_flip[(size_t)c * taps + (taps - 1 - t)] = w_large[e];
        }
    if (role == 2 && g_bu)
        for (int o = tid; o < 9 * Ca; o += nth) {
            float s = 0.f;
#pragma unroll 8
            for (int b = 0; b < B; ++b) s += gdk(b, o);
            g_bu[o] = s;
        }
    if (role == 3 && g_wu)
        for (int e = tid; e < 9 * Ca * hidden; e += nth) {
            const int o = e / hidden, m = e % hidden;
            float s = 0.f;
#pragma unroll 8
            for (int b = 0; b < B; ++b) s = fmaf(gdk(b, o), act[(size_t)b * hidden + m], s);
            g_wu[e] = s;
        }
    if (role == 4 && g_bd)
        for (int m = tid; m < hidden; m += nth) {
            float s = 0.f;
#pragma unroll 8
            for (int b = 0; b < B; ++b) s += gt[(size_t)b * hidden + m];
            g_bd[m] = s;
        }
    if (role == 5 && g_wd)
        for (int e = tid; e < hidden * Ca; e += nth) {
            const int m = e / Ca, k = e % Ca;
            float s = 0.f;
#pragma unroll 8
            for (int b = 0; b < B; ++b) s = fmaf(gt[(size_t)b * hidden + m], gtap[((size_t)b * Ca + k) * kSlot + TAPS] * inv_hw, s);
            g_wd[e] = s;
        }
}

}}  // namespace esc::bwd

// Kernel (a): global average pooling of the attention channels fused with the kernel
// estimator (ESC paper, Section 3.3, Eq. 4 line 2), either reduced to one linear layer
//
//   g[b,c]  = (1/HW) sum_{y,x} x[b,c,y,x]            c < C_a
//   dk[b,o] = b_dyn[o] + sum_c w_dyn[o,c] g[b,c]     o = c*9 + i*3 + j
// or, with hidden > 0, the estimator as Eq. 4 line 2 writes it -- two 1x1 convolutions on the pooled
// vector with the Gaussian error linear unit phi(t) = t * Phi(t) between them:
//   a[b,j]  = phi(b_down[j] + sum_c w_down[j,c] g[b,c])      j < hidden
//   dk[b,o] = b_up[o] + sum_j w_up[o,j] a[b,j]
//
// Every image is cut into S slabs so that a single large image still spreads over the machine;
// the B*S work items are walked by a persistent grid of small blocks (4 warps -- one per SM sub-partition --, at most one block
// per SM).  The blocks are kept this small on purpose: the stencil kernel is launched as a
// programmatic dependent of this one and needs nearly a whole SM per block, so the two kernels
// can only run side by side -- this one bound by DRAM, the other by the FMA pipe -- if this one
// leaves the registers and shared memory free.  A block reduces a slab with 16-byte loads, warp
// shuffles and one pass through shared memory, and writes C_a partial sums.  The block that
// arrives last for an image (a wrapping arrival counter, so no counter ever needs re-zeroing)
// adds the S partial sums in a fixed order -- the result is bitwise reproducible -- and
// evaluates the estimator.
#pragma once
#include "common.cuh"

namespace esc {

constexpr int kGapThreads = 128;
constexpr int kGapWarps = kGapThreads / 32;
constexpr int kMaxHidden = kGapThreads;        // hidden activations live in the block's scratch

// How the block reads an NHWC slab: 16-byte chunks of the attention channels, cpp = C_a / V chunks per
// pixel.  kVecPow2: cpp is a power of two <= 32, lanes with equal lane % cpp hold the same channels and
// a shuffle butterfly adds them.  kVecAny: any other cpp (C_a = 48: six chunks), one row of cpp threads
// per pixel and a reduction through shared memory.  kScalar: channel counts that do not fill chunks.
enum GapRead { kScalar = 0, kVecPow2 = 1, kVecAny = 2 };
__host__ __device__ inline int gap_read_mode(int layout, int C, int Ca, int V) {
    if (layout != kNHWC || Ca % V != 0 || C % V != 0) return kScalar;
    const int cpp = Ca / V;
    if (cpp <= 32 && (cpp & (cpp - 1)) == 0) return kVecPow2;
    return cpp <= kGapThreads ? kVecAny : kScalar;
}
// Floats of block scratch in front of the C_a means.
__host__ __device__ inline int gap_scratch_floats(int layout, int C, int Ca, int V) {
    int n = kGapWarps * Ca > kGapThreads ? kGapWarps * Ca : kGapThreads;
    if (gap_read_mode(layout, C, Ca, V) == kVecAny && kGapThreads * V > n) n = kGapThreads * V;
    return n;
}

// phi(t) = t * Phi(t) with Phi(t) = erfc(-t / sqrt 2) / 2 (no cancellation in the left tail).
__device__ __forceinline__ float gelu_exact(float t) { return 0.5f * t * erfcf(-0.70710678118654752f * t); }

template <typename T, int LAYOUT>
__global__ void __maxnreg__(56)
gap_dynkernel(const T* __restrict__ x, int B, int C, int Ca, int H, int W, int S,
              const T* __restrict__ w_dyn, const T* __restrict__ b_dyn,   // last layer: [9*Ca][n_in], [9*Ca]
              const T* __restrict__ w_down, const T* __restrict__ b_down, // hidden layer [hidden][Ca], [hidden] (hidden > 0)
              int hidden,                      // 0: one linear layer, n_in = Ca; else n_in = hidden
              float* __restrict__ partial,     // [B][S][Ca]
              unsigned* __restrict__ arrivals, // [B]
              float* __restrict__ dk)          // [B][9*Ca]
{
    constexpr int V = Elem<T>::kVec;
    extern __shared__ float smem[];            // gap_scratch_floats() floats of scratch, then [Ca] means
    float* wsum = smem;
    float* gmean = smem + gap_scratch_floats(LAYOUT, C, Ca, V);
    __shared__ bool is_last;

    pdl_launch_dependents();                   // the stencil kernel may start its prologue now

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long HW = (long long)H * W;
    for (int item = blockIdx.x; item < B * S; item += gridDim.x) {
    const int b = item / S, s = item - b * S;
    float* my_partial = partial + ((size_t)b * S + s) * Ca;

    const int cpp = Ca / V;                    // 16-byte chunks per pixel (NHWC)
    const int mode = gap_read_mode(LAYOUT, C, Ca, V);

    if (mode == kVecAny) {
        // Thread t owns chunk t % cpp of pixels t / cpp, t / cpp + ppb, ...; the last 128 % cpp threads idle.
        const long long p0 = HW * s / S, p1 = HW * (s + 1) / S;
        const int chunk = tid % cpp, prow = tid / cpp, ppb = kGapThreads / cpp;
        float acc[V];
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = 0.f;
        if (prow < ppb) {
            const T* base = x + ((size_t)b * HW) * C + (size_t)chunk * V;
            for (long long p = p0 + prow; p < p1; p += 8LL * ppb) {        // eight independent loads in flight
                uint4 q[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const long long pu = p + (long long)u * ppb;
                    q[u] = pu < p1 ? __ldg(reinterpret_cast<const uint4*>(base + (size_t)pu * C)) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    float f[V];
                    unpack16<T>(q[u], f);
#pragma unroll
                    for (int v = 0; v < V; ++v) acc[v] += f[v];
                }
            }
        }
#pragma unroll
        for (int v = 0; v < V; ++v) wsum[tid * V + v] = acc[v];
        __syncthreads();
        for (int c = tid; c < Ca; c += kGapThreads) {                      // rows added in order: reproducible
            const float* col = wsum + (c / V) * V + (c % V);
            float t = 0.f;
            for (int r = 0; r < ppb; ++r) t += col[r * cpp * V];
            my_partial[c] = t;
        }
    } else if (mode == kVecPow2) {
        // Thread t owns chunk (t % cpp) of pixels t/cpp, t/cpp + 256/cpp, ...
        const long long p0 = HW * s / S, p1 = HW * (s + 1) / S;
        const int chunk = tid % cpp, ppb = kGapThreads / cpp;
        float acc[V];
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = 0.f;
        const T* base = x + ((size_t)b * HW) * C + (size_t)chunk * V;
        for (long long p = p0 + tid / cpp; p < p1; p += 8LL * ppb) {   // eight independent loads in flight
            uint4 q[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const long long pu = p + (long long)u * ppb;
                q[u] = pu < p1 ? __ldg(reinterpret_cast<const uint4*>(base + (size_t)pu * C)) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                float f[V];
                unpack16<T>(q[u], f);
#pragma unroll
                for (int v = 0; v < V; ++v) acc[v] += f[v];
            }
        }
        // lanes with equal (lane % cpp) hold the same channels: butterfly over the other lane bits
#pragma unroll
        for (int v = 0; v < V; ++v)
            for (int o = 16; o >= cpp; o >>= 1) acc[v] += __shfl_xor_sync(0xffffffffu, acc[v], o);
        if (lane < cpp) {
#pragma unroll
            for (int v = 0; v < V; ++v) wsum[warp * Ca + lane * V + v] = acc[v];
        }
        __syncthreads();
        for (int c = tid; c < Ca; c += kGapThreads) {
            float t = 0.f;
#pragma unroll
            for (int w = 0; w < kGapWarps; ++w) t += wsum[w * Ca + c];
            my_partial[c] = t;
        }
    } else {
        // One warp per channel (channels warp, warp+8, ...); lanes stride over the slab.
        for (int c = warp; c < Ca; c += kGapWarps) {
            float acc = 0.f;
            if (LAYOUT == kNCHW) {
                const T* plane = x + ((size_t)b * C + c) * HW;
                if (HW % V == 0) {
                    const long long nv = HW / V, v0 = nv * s / S, v1 = nv * (s + 1) / S;
                    const uint4* pv = reinterpret_cast<const uint4*>(plane);
                    float a4[4] = {0.f, 0.f, 0.f, 0.f};
                    long long i = v0 + lane;
                    for (; i + 96 < v1; i += 128) {
                        uint4 q[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) q[u] = __ldg(pv + i + 32 * u);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            float f[V];
                            unpack16<T>(q[u], f);
#pragma unroll
                            for (int v = 0; v < V; ++v) a4[u] += f[v];
                        }
                    }
                    for (; i < v1; i += 32) {
                        float f[V];
                        unpack16<T>(__ldg(pv + i), f);
#pragma unroll
                        for (int v = 0; v < V; ++v) a4[0] += f[v];
                    }
                    acc = (a4[0] + a4[1]) + (a4[2] + a4[3]);
                } else {
                    const long long e0 = HW * s / S, e1 = HW * (s + 1) / S;
                    for (long long i = e0 + lane; i < e1; i += 32) acc += Elem<T>::to_f32(plane[i]);
                }
            } else {
                const long long p0 = HW * s / S, p1 = HW * (s + 1) / S;
                const T* base = x + ((size_t)b * HW) * C + c;
                for (long long p = p0 + lane; p < p1; p += 32) acc += Elem<T>::to_f32(base[(size_t)p * C]);
            }
            acc = warp_sum(acc);
            if (lane == 0) my_partial[c] = acc;
        }
    }

    // ---- arrival: the last block of this image finishes the reduction and the linear layer
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned old = atomicInc(arrivals + b, (unsigned)(S - 1));   // wraps back to 0 by itself
        is_last = (old == (unsigned)(S - 1));
    }
    __syncthreads();
    if (!is_last) continue;
    __threadfence();
    const float inv_hw = 1.0f / (float)HW;
    // S partial sums per channel, added in a fixed two-level order: group j takes slabs j, j+ng, ...
    // (all threads busy, loads independent), then the ng group sums are added in order.
    const int ng = Ca <= kGapThreads / 2 ? kGapThreads / Ca : 1;
    if (ng > 1) {
        float* red = wsum;                                   // [ng][Ca] <= kGapThreads floats; the warp sums are dead
        const int c = tid % Ca, j = tid / Ca;
        if (j < ng) {
            const float* pp = partial + (size_t)b * S * Ca + c;
            float t = 0.f;
            for (int k = j; k < S; k += 8 * ng) {            // eight independent loads, added in order
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = k + u * ng < S ? __ldcg(pp + (size_t)(k + u * ng) * Ca) : 0.f;
#pragma unroll
                for (int u = 0; u < 8; ++u) t += v[u];
            }
            red[j * Ca + c] = t;
        }
        __syncthreads();
        if (tid < Ca) {
            float t = 0.f;
            for (int j2 = 0; j2 < ng; ++j2) t += red[j2 * Ca + tid];
            gmean[tid] = t * inv_hw;
        }
    } else {
        for (int c = tid; c < Ca; c += kGapThreads) {
            const float* pp = partial + (size_t)b * S * Ca + c;
            float t = 0.f;
            for (int k = 0; k < S; ++k) t += __ldcg(pp + (size_t)k * Ca);
            gmean[c] = t * inv_hw;
        }
    }
    __syncthreads();
    const float* vin = gmean;                                // input of the last layer
    int n_in = Ca;
    if (hidden > 0) {
        float* act = wsum;                                   // the warp and group sums are dead
        for (int j = tid; j < hidden; j += kGapThreads) {
            float t = Elem<T>::to_f32(b_down[j]);
            const T* wr = w_down + (size_t)j * Ca;
            for (int c = 0; c < Ca; ++c) t = fmaf(Elem<T>::to_f32(wr[c]), gmean[c], t);
            act[j] = gelu_exact(t);
        }
        __syncthreads();
        vin = act; n_in = hidden;
    }
    for (int o = tid; o < 9 * Ca; o += kGapThreads) {
        float acc = Elem<T>::to_f32(b_dyn[o]);
        const T* wr = w_dyn + (size_t)o * n_in;
        for (int c0 = 0; c0 < n_in; c0 += 16) {              // sixteen independent loads, FMAs in input order
            float wv[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) wv[u] = c0 + u < n_in ? Elem<T>::to_f32(wr[c0 + u]) : 0.f;
#pragma unroll
            for (int u = 0; u < 16; ++u)
                if (c0 + u < n_in) acc = fmaf(wv[u], vin[c0 + u], acc);
        }
        dk[(size_t)b * 9 * Ca + o] = acc;
    }
    __syncthreads();                                         // scratch and flag are reused by the next item
    }
}

}  // namespace esc

// Dense large kernel (ESC paper, Section 3.2: LK in R^{13x13x16x16}; Eq. 4 line 3 with that LK) for NHWC
// bf16 tensors with 16 attention channels, on the tensor cores:
//
//   out[b,n,y,x] = sum_{k,i,j} w_dense[n,k,i,j] x[b,k,y+i-6,x+j-6]  +  sum_{i,j} dk[b,n,i,j] x[b,n,y+i-1,x+j-1]
//
// The first sum is an implicit GEMM, M = pixels, N = 16 output channels, K = 16 input channels x 169 taps.
// For one tap the A operand of a 16-pixel run is simply the 16 x 16-channel block of the staged halo tile
// shifted by that tap (a pixel's 16 channels are its 32 contiguous bytes), so the tile is never unfolded:
// one CTA per SM walks 64x16-pixel output tiles; each of its 16 warps owns one tile row = 4 runs of 16
// pixels x 16 output channels (32 fp32 accumulators per lane) and, per tap, reads its B fragments (one
// 16-byte load from a fragment-ordered weight table in shared memory), then per run its A fragment (two
// 8-byte loads, conflict-free thanks to a permutation of k) and issues two mma.sync.m16n8k16 (bf16 in,
// fp32 accumulate).  The dynamic 3x3 kernel stays depth-wise and in fp32: nine FMAs per output on the
// CUDA cores in the epilogue.  Halo tiles arrive by TMA (zero fill outside the image = the padding) into a
// two-deep ring; results are rounded once to bf16, staged in the consumed tile buffer and written with
// one TMA store per tile.
//
// Roofline note: with N = 16 every A fragment (512 bytes per run and tap) feeds only two MMAs, so the
// kernel needs 1/8 byte of shared-memory bandwidth per multiply-add: at 128 bytes per clock and SM that
// caps it at 1024 MAC/clk/SM whichever tensor-core instruction consumes the fragments.
#pragma once
#include "stencil_generic.cuh"
#include "stencil_tma.cuh"

namespace esc { namespace tma {

namespace dense {
constexpr int TW = 64, TH = 16;                    // output tile
constexpr int THP = TH + K13 - 1;                  // 28 staged rows
constexpr int PITCH = TW + K13 - 1;                // 76 staged pixels per row
constexpr int TILE_BYTES = THP * PITCH * CG * 2;   // 68,096
constexpr int WFRAG_BYTES = K13 * K13 * 32 * 16;   // 86,528: [tap][lane] x 4 words
constexpr int DK_BYTES = ((CG * 9 * 4) + 127) / 128 * 128;
constexpr int kThreads = 512, kWarps = 16;
constexpr int RPW = TH / kWarps;                   // tile rows per warp
constexpr int RUNS = (TW / 16) * RPW;              // runs of 16 pixels per warp
static_assert(TILE_BYTES % 128 == 0, "tile buffers keep 128-byte alignment");
static_assert(TH * TW * CG * 2 <= TILE_BYTES, "the result tile is staged in the consumed input buffer");
static_assert(TH % kWarps == 0 && TW == 64, "tile splits into whole runs per warp; u >> 2 and u & 3 assume four runs per row");
constexpr size_t kSmemBytes = 2 * (size_t)TILE_BYTES + WFRAG_BYTES + DK_BYTES + 128;

struct Params {
    int B, C, H, W;
    int tiles_x, tiles_y;
    long long units;                  // B * tiles_y * tiles_x
    const __nv_bfloat16* w_dense;     // [16][16][13][13]  (output channel, input channel, row, column)
    const float* dk;                  // [B][16][9]
    unsigned* ctrl;                   // status words or nullptr
    int wait_first;                   // 1: nothing may be read before the previous kernel of the stream has finished
};
}  // namespace dense

__global__ void __launch_bounds__(dense::kThreads, 1)
stencil_dense_nhwc_bf16(const __grid_constant__ CUtensorMap map_att, const __grid_constant__ CUtensorMap map_res,
                        const dense::Params p, const CopyJob job)
{
    using namespace dense;
    // The last blocks of the grid copy the identity channels.  They need a whole SM like every block of this
    // launch, so they run where a tile-walking CTA has already finished (the tile count is rarely a multiple
    // of the SM count) or after them, without a launch of their own.
    if (job.blocks != 0 && blockIdx.x >= job.first_block) {
        if (p.wait_first) pdl_wait_primary();              // launched on its own: x may still be in the making
        run_copy_job(job, blockIdx.x - job.first_block, threadIdx.x, dense::kThreads);
        return;
    }
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* tilebuf = smem;                                               // 2 x TILE_BYTES
    uint4* wfrag = reinterpret_cast<uint4*>(smem + 2 * TILE_BYTES);              // [tap][lane]
    float* dks = reinterpret_cast<float*>(smem + 2 * TILE_BYTES + WFRAG_BYTES);  // [tap9][16]
    u64* bars = reinterpret_cast<u64*>(smem + 2 * TILE_BYTES + WFRAG_BYTES + DK_BYTES);
    const uint32_t full0 = smem_u32(bars);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    if (tid == 0) {
        mbar_init(full0, 1); mbar_init(full0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (p.wait_first) pdl_wait_primary();
    pdl_launch_dependents();

    const long long first = blockIdx.x, stride = job.blocks != 0 ? job.first_block : gridDim.x;
    const long long my_units = first < p.units ? (p.units - first + stride - 1) / stride : 0;
    auto coords = [&](long long k, int& b, int& ty, int& tx) {
        unsigned u = (unsigned)(first + k * stride);                             // the host guarantees units < 2^31
        tx = (int)(u % (unsigned)p.tiles_x); u /= (unsigned)p.tiles_x;
        ty = (int)(u % (unsigned)p.tiles_y); b = (int)(u / (unsigned)p.tiles_y);
    };
    auto issue_load = [&](long long k) {                                         // thread 0 only
        int b, ty, tx;
        coords(k, b, ty, tx);
        const int buf = (int)(k & 1);
        mbar_expect_tx(full0 + 8 * buf, TILE_BYTES);
        tma_load_4d(smem_u32(tilebuf + (size_t)buf * TILE_BYTES), &map_att, full0 + 8 * buf, 0, tx * TW - P6, ty * TH - P6, b);
    };
    if (tid == 0 && my_units > 0) issue_load(0);

    // ---- weight table in fragment order (overlaps the first tile load).  The tensor-core instruction sums
    // over k in a fixed lane layout, but which channel a k stands for is free as long as A and B agree:
    // k = 2t + e <-> channel 4t + e, k = 8 + 2t + e <-> channel 4t + 2 + e, so that lane (g, t) needs
    // channels 4t..4t+3 of its pixels (one 8-byte read) and, from B, w[n][4t..4t+3] for n = g and g + 8.
    for (int e = tid; e < K13 * K13 * 32; e += dense::kThreads) {
        const int tap = e >> 5, l = e & 31, gg = l >> 2, tt = l & 3;
        const unsigned short* w = reinterpret_cast<const unsigned short*>(p.w_dense) + tap;   // + (n*16 + k) * 169
        unsigned v[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int n = gg + (q >> 2) * 8, k = 4 * tt + (q & 3);
            v[q] = __ldg(w + (size_t)(n * CG + k) * (K13 * K13));
        }
        wfrag[e] = make_uint4(v[0] | (v[1] << 16), v[2] | (v[3] << 16), v[4] | (v[5] << 16), v[6] | (v[7] << 16));
    }
    __syncthreads();

    bool alive = true, dk_ready = p.wait_first != 0;
    int staged_b = -1;
    for (long long k = 0; k < my_units; ++k) {
        int b, ty, tx;
        coords(k, b, ty, tx);
        const int buf = (int)(k & 1);
        unsigned char* tbuf = tilebuf + (size_t)buf * TILE_BYTES;
        if (alive) alive = mbar_wait(full0 + 8 * buf, (unsigned)((k >> 1) & 1), p.ctrl, 0xE0000000u | (unsigned)buf);

        float d[RUNS][2][4];
#pragma unroll
        for (int u = 0; u < RUNS; ++u)
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int e = 0; e < 4; ++e) d[u][h][e] = 0.f;

        // lane's first pixel of run u for tap (0,0): staged row RPW*warp + (u >> 2), staged column 16*(u & 3) + g
        const uint2* a2 = reinterpret_cast<const uint2*>(tbuf) + ((RPW * warp) * PITCH + g) * 4 + t;
#pragma unroll 1
        for (int i = 0; i < K13; ++i) {
            if (i == 1 && tid == 0 && k + 1 < my_units) {
                // the other buffer held the previous tile's result: its store must have read it
                bulk_wait_read<0>();
                issue_load(k + 1);
            }
            const uint2* arow = a2 + i * (PITCH * 4);
            const uint4* wrow = wfrag + (i * K13) * 32 + lane;
#pragma unroll
            for (int j = 0; j < K13; ++j) {
                const uint4 bw = wrow[j * 32];
                const uint32_t b0[2] = {bw.x, bw.y}, b1[2] = {bw.z, bw.w};
#pragma unroll
                for (int u = 0; u < RUNS; ++u) {
                    const uint2* pa = arow + (((u >> 2) * PITCH) + (u & 3) * 16 + j) * 4;
                    const uint2 va = pa[0], vb = pa[8 * 4];
                    const uint32_t a[4] = {va.x, vb.x, va.y, vb.y};
                    mma_16x8x16_bf16(d[u][0], a, b0);
                    mma_16x8x16_bf16(d[u][1], a, b1);
                }
            }
        }

        // ---- dynamic 3x3 kernel, depth-wise, fp32 (Eq. 4 line 3, second term) ----------------------------
        if (staged_b != b) {
            if (!dk_ready) { pdl_wait_primary(); dk_ready = true; }
            if (tid < CG * 9) dks[(tid % 9) * CG + tid / 9] = __ldcg(p.dk + (size_t)b * CG * 9 + tid);
            staged_b = b;
        }
        __syncthreads();                                     // dk staged
        {
            // lane holds, per run, pixels g and g+8 x channels {2t, 2t+1} (d[u][0]) and {8+2t, 9+2t} (d[u][1])
            const uint32_t* x32 = reinterpret_cast<const uint32_t*>(tbuf);
#pragma unroll
            for (int tap = 0; tap < 9; ++tap) {
                const float2 k0 = *reinterpret_cast<const float2*>(dks + tap * CG + 2 * t);
                const float2 k1 = *reinterpret_cast<const float2*>(dks + tap * CG + 8 + 2 * t);
                const int off = ((P6 - 1 + tap / 3) * PITCH + (P6 - 1 + tap % 3)) * NPAIR;
#pragma unroll
                for (int u = 0; u < RUNS; ++u) {
                    const int px = ((RPW * warp + (u >> 2)) * PITCH + (u & 3) * 16 + g) * NPAIR + off;
#pragma unroll
                    for (int r = 0; r < 2; ++r) {            // pixel g, pixel g + 8
                        const uint32_t v0 = x32[px + r * 8 * NPAIR + t], v1 = x32[px + r * 8 * NPAIR + 4 + t];
                        d[u][0][2 * r] = fmaf(k0.x, __uint_as_float(v0 << 16), d[u][0][2 * r]);
                        d[u][0][2 * r + 1] = fmaf(k0.y, __uint_as_float(v0 & 0xffff0000u), d[u][0][2 * r + 1]);
                        d[u][1][2 * r] = fmaf(k1.x, __uint_as_float(v1 << 16), d[u][1][2 * r]);
                        d[u][1][2 * r + 1] = fmaf(k1.y, __uint_as_float(v1 & 0xffff0000u), d[u][1][2 * r + 1]);
                    }
                }
            }
        }
        __syncthreads();                                     // every warp has finished reading this tile

        // ---- round once to bf16, stage the 16 x 64 x 16 result in the consumed buffer, one TMA store ------
        {
            uint32_t* s32 = reinterpret_cast<uint32_t*>(tbuf);
#pragma unroll
            for (int u = 0; u < RUNS; ++u) {
                const int px = ((RPW * warp + (u >> 2)) * TW + (u & 3) * 16 + g) * NPAIR;
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    s32[px + r * 8 * NPAIR + t] = pack_bf16x2(d[u][0][2 * r], d[u][0][2 * r + 1]);
                    s32[px + r * 8 * NPAIR + 4 + t] = pack_bf16x2(d[u][1][2 * r], d[u][1][2 * r + 1]);
                }
            }
        }
        fence_async_smem();
        __syncthreads();
        if (tid == 0) {
            tma_store_4d(&map_res, smem_u32(tbuf), 0, tx * TW, ty * TH, b);
            bulk_commit();
        }
    }
    if (tid == 0) bulk_wait_all<0>();
}

// One thread per output for every other element type, layout or channel count: correct everywhere, slow.
template <typename T, int LAYOUT>
__global__ void __launch_bounds__(256)
stencil_dense_generic(const T* __restrict__ x, T* __restrict__ out, int B, int C, int Ca, int H, int W, int K,
                      const T* __restrict__ w_dense, const float* __restrict__ dk)
{
    pdl_wait_primary();
    const int P = (K - 1) / 2;
    const long long total = (long long)B * Ca * H * W;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        long long r = e;
        int xx, y, n, b;
        if (LAYOUT == kNHWC) { n = (int)(r % Ca); r /= Ca; xx = (int)(r % W); r /= W; y = (int)(r % H); b = (int)(r / H); }
        else { xx = (int)(r % W); r /= W; y = (int)(r % H); r /= H; n = (int)(r % Ca); b = (int)(r / Ca); }
        float acc = 0.f;
        for (int k = 0; k < Ca; ++k)
            for (int i = 0; i < K; ++i) {
                const int yy = y + i - P;
                if (yy < 0 || yy >= H) continue;
                for (int j = 0; j < K; ++j) {
                    const int xc = xx + j - P;
                    if (xc < 0 || xc >= W) continue;
                    acc = fmaf(Elem<T>::to_f32(w_dense[(((size_t)n * Ca + k) * K + i) * K + j]),
                               Elem<T>::to_f32(x[elem_index<LAYOUT>(b, k, yy, xc, C, H, W)]), acc);
                }
            }
        for (int i = 0; i < 3; ++i)
            for (int j = 0; j < 3; ++j) {
                const int yy = y + i - 1, xc = xx + j - 1;
                if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                    acc = fmaf(dk[((size_t)b * Ca + n) * 9 + i * 3 + j], Elem<T>::to_f32(x[elem_index<LAYOUT>(b, n, yy, xc, C, H, W)]), acc);
            }
        out[elem_index<LAYOUT>(b, n, y, xx, C, H, W)] = Elem<T>::from_f32(acc);
    }
}

// Launches the tensor-core kernel if the problem fits it (K = 13, bf16, NHWC, 16 attention channels).
// Returns 0, kNotApplicable, or an ESC_ERR_* code.
inline int try_launch_dense(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x,
                            const void* w_dense, const float* dk, void* out, unsigned* ctrl, cudaStream_t st,
                            bool dependent, CopyJob job, int* launches, std::string* err) {
    using namespace dense;
    if (K != K13 || dtype != 1 /*bf16*/ || layout != kNHWC || Ca != CG || C % 8 != 0) return kNotApplicable;
    if ((reinterpret_cast<uintptr_t>(w_dense) & 1) != 0) return kNotApplicable;
    const int sms = sm_count();
    if (sms <= 0) return kNotApplicable;
    dense::Params p;
    p.B = B; p.C = C; p.H = H; p.W = W;
    p.tiles_x = (W + TW - 1) / TW; p.tiles_y = (H + TH - 1) / TH;
    p.units = (long long)B * p.tiles_x * p.tiles_y;
    if (p.units > 0x7fffffffLL) return kNotApplicable;
    p.w_dense = static_cast<const __nv_bfloat16*>(w_dense);
    p.dk = dk;
    p.ctrl = ctrl;
    p.wait_first = dependent ? 0 : 1;
    CUtensorMap m_att, m_res;
    if (!make_map(&m_att, x, B, C, H, W, CG, PITCH, THP, CU_TENSOR_MAP_L2_PROMOTION_L2_64B)) return kNotApplicable;
    if (!make_map(&m_res, out, B, C, H, W, CG, TW, TH)) return kNotApplicable;
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return kNotApplicable;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(stencil_dense_nhwc_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return kNotApplicable; }
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    const unsigned walkers = (unsigned)(p.units < sms ? p.units : sms);
    if (job.blocks != 0) job.first_block = walkers;
    cfg.gridDim = dim3(walkers + job.blocks);
    cfg.blockDim = dim3(dense::kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, stencil_dense_nhwc_bf16, m_att, m_res, p, job);
    if (e != cudaSuccess) {
        char buf[256];
        snprintf(buf, sizeof buf, "stencil_dense_nhwc_bf16 launch: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e));
        *err = buf;
        return 7;  // ESC_ERR_CUDA
    }
    ++*launches;
    return 0;
}

}}  // namespace esc::tma

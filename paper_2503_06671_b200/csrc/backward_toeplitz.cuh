// Per-tile tap gradients of the ConvAttn backward pass (ESC paper, Section 3.3, Eq. 4 line 3, differentiated with
// respect to the taps) on the tensor cores, for NHWC bf16 tensors with whole groups of 16 attention channels:
//
//   g_tap[b,c,i,j] = sum_{y,x} go[b,c,y,x] * x~[b,c,y+i-6,x+j-6]          (x~: x with zero padding)
//
// For one row y of a tile of go and a kernel row i the 13 sums over x are a product with a banded Toeplitz matrix
// built from the go row:  D[j][i] += sum_u G_y[j][u] * X[u][i],  G_y[j][u] = go[y][u - j],  X[u][i] = x~[y + i][u]
// (u = x + j: the staged column).  One tensor-core instruction (16 x 8 x 16) takes 16 staged columns, all 13 (of 16)
// tap columns j and 8 kernel rows i: 13 x 13 of 16 x 16 multiply-adds are useful, the image operand comes straight
// from the channel's plane by ldmatrix, and the Toeplitz operand's registers are pairs (go[d], go[d + 1]) read from the
// go plane (two aligned words and a funnel shift where d is odd).  bf16 products are exact in fp32 and accumulation
// is fp32: the arithmetic of the FP32 kernel (tap_grad_nhwc8) in another order.
//
// One CTA per SM, persistent over units (a 64 x 16 tile of go, its 76 x 28 halo tile of x, 16 channels):
//   warp 8     lane 0 requests both tiles by TMA (zero fill = the padding)
//   warps 0-7  transpose both tiles into per-channel planes (as the forward kernel does), then two channels each:
//              16 rows x 5 column blocks x 2 instructions; 169 sums and the sum of the tile's x values per channel go
//              to the tile's slot of the workspace, which sum_tiles and finish (backward.cuh) consume.
#pragma once
#include "backward.cuh"
#include "stencil_toeplitz.cuh"

namespace esc { namespace bwd { namespace toep {

using tma::CG; using tma::K13; using tma::P6; using tma::u64; using tma::Unit;
using tma::toep::ldsm_x4; using tma::toep::ldsm_x4_trans; using tma::toep::mma_bf16; using tma::toep::mma_bar;
using S = tma::toep::Shape64x16;
constexpr int kWarps = 8, kThreads = kWarps * 32 + 32;
constexpr int TH = S::TH, TW = S::TW, ROWS = S::ROWS, SW = S::SW, PP = S::PP, PLANE = S::PLANE_BYTES;
constexpr int GP = TW + 16;                               // go plane row: 8 zeros, 64 values, 8 zeros
constexpr int GPLANE = TH * GP * 2 + 80;                  // 2,640 bytes = 660 words = 20 (mod 32): the transposition's stores spread over the banks
constexpr int STAGE_X = S::STAGE_BYTES, STAGE_G = S::BOX_BYTES;
constexpr size_t kSmemBytes = (size_t)STAGE_X + STAGE_G + CG * PLANE + CG * GPLANE + 64;
static_assert(STAGE_X % 128 == 0 && STAGE_G % 128 == 0 && (GPLANE / 4) % 32 == 20 && kSmemBytes <= 227 * 1024, "layout");

struct Params {
    int B, C, Ca, H, W;
    int tiles_x, tiles_y, groups;
    long long units;
    float* part;                      // [B][Ca][tiles][kSlot]
    unsigned* ctrl;
};

__device__ __forceinline__ Unit decode(long long u64v, const Params& p) {
    unsigned u = (unsigned)u64v;
    Unit r;
    r.tx = (int)(u % (unsigned)p.tiles_x); u /= (unsigned)p.tiles_x;
    r.ty = (int)(u % (unsigned)p.tiles_y); u /= (unsigned)p.tiles_y;
    r.g = (int)(u % (unsigned)p.groups);
    r.b = (int)(u / (unsigned)p.groups);
    return r;
}

__global__ void __launch_bounds__(kThreads, 1)
tap_grad_toeplitz_nhwc_bf16(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_go, const Params p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* stage_x = smem;                                 // x halo tile as it lands: [ROWS][SW][16] bf16
    unsigned char* stage_g = smem + STAGE_X;                       // go tile as it lands: [TH][TW][16] bf16
    unsigned char* xpl = stage_g + STAGE_G;                        // 16 x [ROWS][PP] bf16
    unsigned char* gpl = xpl + CG * PLANE;                         // 16 x [TH][GP] bf16 (+ padding)
    u64* bars = reinterpret_cast<u64*>(gpl + CG * GPLANE);
    const uint32_t full = tma::smem_u32(bars), empty = full + 8;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        tma::mbar_init(full, 1);
        tma::mbar_init(empty, kWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // the zero borders of the go planes are written once; the transposition touches columns 8 .. 71 only
    for (int e = tid; e < CG * TH * 8; e += kThreads) {
        const int c = e / (TH * 8), r = (e / 8) % TH, q = e % 8;   // eight words per row: four on either side
        uint32_t* row = reinterpret_cast<uint32_t*>(gpl + (size_t)c * GPLANE + (size_t)r * GP * 2);
        row[q < 4 ? q : (GP / 2 - 8 + q)] = 0u;
    }
    __syncthreads();

    const long long first = blockIdx.x, stride = gridDim.x;
    const long long my_units = first < p.units ? (p.units - first + stride - 1) / stride : 0;

    if (warp == kWarps) {
        if (lane != 0) return;
        bool alive = true;
        for (long long k = 0; k < my_units; ++k) {
            if (k >= 1 && alive) alive = tma::mbar_wait(empty, (unsigned)((k - 1) & 1), p.ctrl, 0xD8000000u);
            const Unit un = decode(first + k * stride, p);
            tma::mbar_expect_tx(full, STAGE_X + STAGE_G);
            tma::tma_load_4d(tma::smem_u32(stage_x), &map_x, full, un.g * CG, un.tx * TW - P6, un.ty * TH - P6, un.b);
            tma::tma_load_4d(tma::smem_u32(stage_g), &map_go, full, un.g * CG, un.tx * TW, un.ty * TH, un.b);
        }
        return;
    }

    const int g = lane >> 2, t = lane & 3;
    const int mi = lane >> 3, mr = lane & 7;
    const uint32_t xpl_a = tma::smem_u32(xpl);
    const int tiles = p.tiles_x * p.tiles_y;
    bool alive = true;

    for (long long k = 0; k < my_units; ++k) {
        const Unit un = decode(first + k * stride, p);
        if (alive) alive = tma::mbar_wait(full, (unsigned)(k & 1), p.ctrl, 0xD9000000u);
        // ---- transpose both tiles into per-channel planes: 16 pixels x 16 channels per step ------------------------
        {
            const uint32_t lane_off = (uint32_t)(((mi >> 1) * 8 + mr) * (CG * 2) + (mi & 1) * 16);
            const uint32_t sx = tma::smem_u32(stage_x) + lane_off, sg = tma::smem_u32(stage_g) + lane_off;
            for (int s = warp; s < ROWS * (SW / 16); s += kWarps) {
                const int row = s / (SW / 16), x0 = (s % (SW / 16)) * 16;
                uint32_t r[4];
                ldsm_x4_trans(sx + (uint32_t)((row * SW + x0) * (CG * 2)), r);
                // r[j], lane (g, t): channel 8 * (j & 1) + g, pixels x0 + 8 * (j >> 1) + 2t, + 1
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int c = 8 * (j & 1) + g, x = x0 + 8 * (j >> 1) + 2 * t;
                    *reinterpret_cast<uint32_t*>(xpl + (size_t)c * PLANE + ((size_t)row * PP + x) * 2) = r[j];
                }
            }
            for (int s = warp; s < TH * (TW / 16); s += kWarps) {
                const int row = s / (TW / 16), x0 = (s % (TW / 16)) * 16;
                uint32_t r[4];
                ldsm_x4_trans(sg + (uint32_t)((row * TW + x0) * (CG * 2)), r);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int c = 8 * (j & 1) + g, x = 8 + x0 + 8 * (j >> 1) + 2 * t;
                    *reinterpret_cast<uint32_t*>(gpl + (size_t)c * GPLANE + ((size_t)row * GP + x) * 2) = r[j];
                }
            }
        }
        __syncwarp();
        if (lane == 0) tma::mbar_arrive(empty);              // both staging buffers may be refilled
        mma_bar();                                           // the planes are complete

        const int tile = un.ty * p.tiles_x + un.tx;
        const unsigned sh = (g & 1) ? 16u : 0u;              // d = 16 ub + 2t - g is odd where g is: the pair straddles two words
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
            const int c = warp * 2 + cc;
            float* slot = p.part + (((size_t)un.b * p.Ca + un.g * CG + c) * tiles + tile) * kSlot;
            // ---- the sum of the tile's x values (the pooled mean is recomputed from it): a row of 64 pixels per load ----
            {
                const uint32_t* pl = reinterpret_cast<const uint32_t*>(xpl + (size_t)c * PLANE) + (P6 * PP + P6) / 2 + lane;
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int r = 0; r < TH; ++r) {
                    const uint32_t v = pl[r * (PP / 2)];
                    s0 += __uint_as_float(v << 16);
                    s1 += __uint_as_float(v & 0xffff0000u);
                }
                float s = s0 + s1;
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                if (lane == 0) slot[TAPS] = s;
            }
            // ---- D[j][i]: rows j = g, g + 8; columns i = 2t, 2t + 1 (d0) and 8 + 2t, 9 + 2t (d1) ----------------------
            float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t* gw = reinterpret_cast<const uint32_t*>(gpl + (size_t)c * GPLANE);
            const int w0 = (8 + 2 * t - g) >> 1;             // word of staged go column d = 2t - g (stored at d + 8); >= 0
#pragma unroll 2
            for (int y = 0; y < TH; ++y) {
                // image operand: matrix mi = (kernel-row half, column half); rows beyond the staged 28 belong to i >= 13
                const int xr = min(y + (mi >> 1) * 8 + mr, ROWS - 1);
                const uint32_t b_lane = xpl_a + (uint32_t)c * PLANE + (uint32_t)((xr * PP + (mi & 1) * 8) * 2);
                const uint32_t* gr = gw + y * (GP / 2) + w0;
                uint32_t a_prev = 0u;                        // P[16 ub + e - 8]: all its columns are left of the tile for ub = 0
#pragma unroll
                for (int ub = 0; ub < SW / 16; ++ub) {
                    uint32_t b[4];
                    ldsm_x4(b_lane + (uint32_t)(16 * ub * 2), b);
                    const uint32_t a0 = __funnelshift_r(gr[8 * ub], gr[8 * ub + 1], sh);
                    // P[16 ub + e + 8]: beyond the tile's last column for the last block
                    const uint32_t a2 = ub + 1 < SW / 16 ? __funnelshift_r(gr[8 * ub + 4], gr[8 * ub + 5], sh) : 0u;
                    mma_bf16(d0, a0, a_prev, a2, a0, b[0], b[1]);
                    mma_bf16(d1, a0, a_prev, a2, a0, b[2], b[3]);
                    a_prev = a2;
                }
            }
            // ---- 13 x 13 of the 16 x 16 sums are taps ----------------------------------------------------------
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int j = g + 8 * h;
                if (j < K13) {
                    const int i0 = 2 * t, i1 = 8 + 2 * t;
                    slot[i0 * K13 + j] = d0[2 * h];
                    slot[(i0 + 1) * K13 + j] = d0[2 * h + 1];
                    if (i1 < K13) slot[i1 * K13 + j] = d1[2 * h];
                    if (i1 + 1 < K13) slot[(i1 + 1) * K13 + j] = d1[2 * h + 1];
                }
            }
        }
        mma_bar();                                           // the planes are free for the next unit
    }
}

inline bool applies(int C, int Ca, int K, int dtype, int layout, const void* x, const void* go) {
    return K == K13 && dtype == 1 /*bf16*/ && layout == kNHWC && Ca % CG == 0 && C % 8 == 0 &&
           (reinterpret_cast<uintptr_t>(x) & 15u) == 0 && (reinterpret_cast<uintptr_t>(go) & 15u) == 0;
}
inline int tiles_of(int H, int W) { return ((W + TW - 1) / TW) * ((H + TH - 1) / TH); }

// 0 on success, tma::kNotApplicable where the kernel does not take the problem, else an ESC_ERR_* code.
inline int try_launch(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x, const void* go,
                      float* part, unsigned* ctrl, cudaStream_t st, int* launches, std::string* err) {
    if (!applies(C, Ca, K, dtype, layout, x, go) || tma::sm_count() <= 0) return tma::kNotApplicable;
    Params p;
    p.B = B; p.C = C; p.Ca = Ca; p.H = H; p.W = W;
    p.tiles_x = (W + TW - 1) / TW; p.tiles_y = (H + TH - 1) / TH; p.groups = Ca / CG;
    p.units = (long long)B * p.groups * p.tiles_x * p.tiles_y;
    if (p.units > 0x7fffffffLL) return tma::kNotApplicable;
    p.part = part; p.ctrl = ctrl;
    CUtensorMap m_x, m_go;
    if (!tma::make_map(&m_x, x, B, C, H, W, CG, SW, ROWS, CU_TENSOR_MAP_L2_PROMOTION_L2_64B)) return tma::kNotApplicable;
    if (!tma::make_map(&m_go, go, B, C, H, W, CG, TW, TH, CU_TENSOR_MAP_L2_PROMOTION_L2_64B)) return tma::kNotApplicable;
    static bool attr_set[tma::kMaxDevices] = {};
    const int dev = tma::current_device();
    if (dev < 0) return tma::kNotApplicable;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tap_grad_toeplitz_nhwc_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return tma::kNotApplicable; }
        attr_set[dev] = true;
    }
    const long long grid = p.units < tma::sm_count() ? p.units : tma::sm_count();
    tap_grad_toeplitz_nhwc_bf16<<<(unsigned)grid, kThreads, kSmemBytes, st>>>(m_x, m_go, p);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        char buf[256];
        snprintf(buf, sizeof buf, "tap_grad_toeplitz_nhwc_bf16 launch: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e));
        *err = buf;
        return 7;  // ESC_ERR_CUDA
    }
    ++*launches;
    return 0;
}

}}}  // namespace esc::bwd::toep

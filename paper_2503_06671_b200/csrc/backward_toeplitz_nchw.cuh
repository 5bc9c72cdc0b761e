// Per-tile tap gradients of the ConvAttn backward pass on the tensor cores for NCHW bf16 tensors: the arithmetic of
// backward_toeplitz.cuh on the layout whose rows are already x-contiguous per channel (ESC paper, Section 3.3, Eq. 4
// line 3, differentiated with respect to the taps):
//
//   g_tap[b,c,i,j] = sum_{y,x} go[b,c,y,x] * x~[b,c,y+i-6,x+j-6]
//   D[j][i] += sum_s G_y[j][s] * X[s][i],   G_y[j][s] = go[y][s - j - 2],   X[s][i] = x~[y + i][s]   (s: staged column)
//
// Both tiles land by TMA directly as the per-channel planes the instruction reads -- x: 16 channels x 28 rows x 88
// columns from 8 columns left of the tile (a TMA load starts on a 16-byte boundary; the Toeplitz band of go is shifted
// by two columns instead), go: 16 x 16 x 88 from 16 columns left of it.  The go plane therefore holds the neighbouring
// tiles' values where the NHWC kernel has zeros: the four register pairs that can reach them (first and last column
// block) are masked with per-lane constants.  x tiles are double-buffered; the go tile is loaded when the warps are
// done with the previous one.  No block-wide barrier: buffers are handed over through mbarriers, warp by warp.
#pragma once
#include "backward_toeplitz.cuh"
#include "stencil_toeplitz_nchw.cuh"

namespace esc { namespace bwd { namespace toepn {

using tma::CG; using tma::K13; using tma::P6; using tma::u64; using tma::Unit;
using tma::toep::ldsm_x4; using tma::toep::mma_bf16;
constexpr int kWarps = 8, kThreads = kWarps * 32 + 32;
constexpr int TH = tma::toepn::TH, TW = tma::toepn::TW, ROWS = tma::toepn::ROWS, PP = tma::toepn::PP, XS = tma::toepn::XS;
constexpr int PLANE = tma::toepn::PLANE, XBUF = tma::toepn::BUF_BYTES;
constexpr int GS = 16;                                    // go columns staged left of the tile (a multiple of 8)
constexpr int GP = 88;                                    // staged go columns = plane row pitch
constexpr int GPLANE = TH * GP * 2, GBUF = CG * GPLANE;   // 2,816 / 45,056 bytes
constexpr int NUB = 5;                                    // column blocks of 16 staged x columns that meet the tile's taps
constexpr size_t kSmemBytes = (size_t)2 * XBUF + GBUF + 64;
static_assert(XBUF % 128 == 0 && GBUF % 128 == 0 && kSmemBytes <= 227 * 1024, "layout");
static_assert(16 * NUB + 8 <= PP && GS + TW + 8 <= GP, "operands stay inside their plane rows");

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
tap_grad_toeplitz_nchw_bf16(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_go, const Params p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* xbufs = smem;                                   // 2 x 16 planes [ROWS][PP] bf16
    unsigned char* gbuf = smem + 2 * XBUF;                         // 16 planes [TH][GP] bf16
    u64* bars = reinterpret_cast<u64*>(gbuf + GBUF);
    const uint32_t xfull0 = tma::smem_u32(bars), xempty0 = xfull0 + 16, gfull = xempty0 + 16, gempty = gfull + 8;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < 2; ++s) { tma::mbar_init(xfull0 + 8 * s, 1); tma::mbar_init(xempty0 + 8 * s, kWarps); }
        tma::mbar_init(gfull, 1);
        tma::mbar_init(gempty, kWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const long long first = blockIdx.x, stride = gridDim.x;
    const long long my_units = first < p.units ? (p.units - first + stride - 1) / stride : 0;

    if (warp == kWarps) {
        if (lane != 0) return;
        bool alive = true;
        for (long long k = 0; k < my_units; ++k) {
            const int buf = (int)(k & 1);
            const Unit un = decode(first + k * stride, p);
            if (k >= 2 && alive) alive = tma::mbar_wait(xempty0 + 8 * buf, (unsigned)(((k >> 1) - 1) & 1), p.ctrl, 0xDA000000u);
            tma::mbar_expect_tx(xfull0 + 8 * buf, XBUF);
            tma::tma_load_4d(tma::smem_u32(xbufs + buf * XBUF), &map_x, xfull0 + 8 * buf, un.tx * TW - XS, un.ty * TH - P6, un.g * CG, un.b);
            if (k >= 1 && alive) alive = tma::mbar_wait(gempty, (unsigned)((k - 1) & 1), p.ctrl, 0xDB000000u);
            tma::mbar_expect_tx(gfull, GBUF);
            tma::tma_load_4d(tma::smem_u32(gbuf), &map_go, gfull, un.tx * TW - GS, un.ty * TH, un.g * CG, un.b);
        }
        return;
    }

    const int g = lane >> 2, t = lane & 3;
    const int mi = lane >> 3, mr = lane & 7;
    const int tiles = p.tiles_x * p.tiles_y;
    // A pair (go[d], go[d + 1]) of column block ub starts at d = 16 ub + e; e = 2t - g - 2 (the x tile starts 8, not 6,
    // columns left of the tile).  Stored at column d + GS; d is odd where g is, then the pair straddles two words.
    const int e = 2 * t - g - (XS - P6);
    const unsigned sh = (g & 1) ? 16u : 0u;
    const int w0 = (GS + e) >> 1;                            // word of the pair of block 0; >= 3
    // Columns outside 0 .. TW-1 of the go plane belong to neighbouring tiles: the pairs of the first and last block
    // that can reach them are masked.  valid(d) = 0 <= d < TW.
    auto pair_mask = [](int d) -> uint32_t {
        return ((d >= 0 && d < TW) ? 0x0000ffffu : 0u) | ((d + 1 >= 0 && d + 1 < TW) ? 0xffff0000u : 0u);
    };
    const uint32_t m_a0_first = pair_mask(e), m_a2_first = pair_mask(e + 8);
    const uint32_t m_a0_last = pair_mask(16 * (NUB - 1) + e), m_a2_last = pair_mask(16 * (NUB - 1) + e + 8);
    bool alive = true;

    for (long long k = 0; k < my_units; ++k) {
        const Unit un = decode(first + k * stride, p);
        const int buf = (int)(k & 1);
        const unsigned char* xpl = xbufs + buf * XBUF;
        if (alive) alive = tma::mbar_wait(xfull0 + 8 * buf, (unsigned)((k >> 1) & 1), p.ctrl, 0xDC000000u);
        if (alive) alive = tma::mbar_wait(gfull, (unsigned)(k & 1), p.ctrl, 0xDD000000u);
        const int tile = un.ty * p.tiles_x + un.tx;
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
            const int c = warp * 2 + cc;
            float* slot = p.part + (((size_t)un.b * p.Ca + un.g * CG + c) * tiles + tile) * kSlot;
            // ---- the sum of the tile's x values: a row of 64 pixels per load ------------------------------------
            {
                const uint32_t* pl = reinterpret_cast<const uint32_t*>(xpl + (size_t)c * PLANE) + (P6 * PP + XS) / 2 + lane;
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
            const uint32_t* gw = reinterpret_cast<const uint32_t*>(gbuf + (size_t)c * GPLANE);
            const uint32_t xpl_a = tma::smem_u32(xpl) + (uint32_t)c * PLANE;
#pragma unroll 2
            for (int y = 0; y < TH; ++y) {
                // image operand: matrix mi = (kernel-row half, column half); rows beyond the staged 28 belong to i >= 13
                const int xr = min(y + (mi >> 1) * 8 + mr, ROWS - 1);
                const uint32_t b_lane = xpl_a + (uint32_t)((xr * PP + (mi & 1) * 8) * 2);
                const uint32_t* gr = gw + y * (GP / 2) + w0;
                uint32_t a_prev = 0u;                        // P[e - 8]: every column is left of the tile
#pragma unroll
                for (int ub = 0; ub < NUB; ++ub) {
                    uint32_t b[4];
                    ldsm_x4(b_lane + (uint32_t)(16 * ub * 2), b);
                    uint32_t a0 = __funnelshift_r(gr[8 * ub], gr[8 * ub + 1], sh);
                    uint32_t a2 = __funnelshift_r(gr[8 * ub + 4], gr[8 * ub + 5], sh);
                    if (ub == 0) { a0 &= m_a0_first; a2 &= m_a2_first; }
                    if (ub == NUB - 1) { a0 &= m_a0_last; a2 &= m_a2_last; }
                    mma_bf16(d0, a0, a_prev, a2, a0, b[0], b[1]);
                    mma_bf16(d1, a0, a_prev, a2, a0, b[2], b[3]);
                    a_prev = a2;
                }
            }
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
        __syncwarp();
        if (lane == 0) { tma::mbar_arrive(xempty0 + 8 * buf); tma::mbar_arrive(gempty); }
    }
}

inline int make_map_go(CUtensorMap* m, const void* base, int B, int C, int H, int W) {
    tma::EncodeTiledFn fn = tma::encode_fn();
    if (!fn) return 0;
    const cuuint64_t dims[4] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)C, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)W * 2, (cuuint64_t)H * W * 2, (cuuint64_t)C * H * W * 2};
    const cuuint32_t box[4] = {(cuuint32_t)GP, (cuuint32_t)TH, (cuuint32_t)CG, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 0 on success, tma::kNotApplicable where the kernel does not take the problem, else an ESC_ERR_* code.
inline int try_launch(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x, const void* go,
                      float* part, unsigned* ctrl, cudaStream_t st, int* launches, std::string* err) {
    if (!tma::toepn::applies(C, Ca, H, W, K, dtype, layout, x, go) || tma::sm_count() <= 0) return tma::kNotApplicable;
    Params p;
    p.B = B; p.C = C; p.Ca = Ca; p.H = H; p.W = W;
    p.tiles_x = (W + TW - 1) / TW; p.tiles_y = (H + TH - 1) / TH; p.groups = Ca / CG;
    p.units = (long long)B * p.groups * p.tiles_x * p.tiles_y;
    if (p.units > 0x7fffffffLL) return tma::kNotApplicable;
    p.part = part; p.ctrl = ctrl;
    CUtensorMap m_x, m_go;
    if (!tma::toepn::make_map_nchw(&m_x, x, B, C, H, W)) return tma::kNotApplicable;
    if (!make_map_go(&m_go, go, B, C, H, W)) return tma::kNotApplicable;
    static bool attr_set[tma::kMaxDevices] = {};
    const int dev = tma::current_device();
    if (dev < 0) return tma::kNotApplicable;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tap_grad_toeplitz_nchw_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return tma::kNotApplicable; }
        attr_set[dev] = true;
    }
    const long long grid = p.units < tma::sm_count() ? p.units : tma::sm_count();
    tap_grad_toeplitz_nchw_bf16<<<(unsigned)grid, kThreads, kSmemBytes, st>>>(m_x, m_go, p);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        char buf[256];
        snprintf(buf, sizeof buf, "tap_grad_toeplitz_nchw_bf16 launch: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e));
        *err = buf;
        return 7;  // ESC_ERR_CUDA
    }
    ++*launches;
    return 0;
}

}}}  // namespace esc::bwd::toepn

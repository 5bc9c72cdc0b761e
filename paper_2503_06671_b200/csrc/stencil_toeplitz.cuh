// Kernel (b), tensor-core form: the K = 13 depth-wise stage of ConvAttn on NHWC bf16 tensors as
// banded-Toeplitz matrix products (ESC paper, Section 3.3, Eq. 4 lines 3-4).
//
// A depth-wise convolution is not a dense contraction over channels, but along one image axis it
// is one: for a channel c and a kernel row i
//     out[y][x] += sum_xin  T_i[x][xin] * in[y + i][xin],     T_i[x][xin] = LK[c][i][xin - x]  (0 <= xin - x < 13),
// a product of a banded Toeplitz matrix of weights with a block of the image.  With 16 outputs per
// row block the band needs 28 inputs, i.e. two k-steps of the 16x8x16 tensor-core instruction:
// 13 of every 32 multiply-adds are useful, and the instruction is still three times faster than the
// FP32 pipe at its peak (bf16 products are exact in fp32, accumulation is fp32, so the arithmetic
// is the one the FP32 kernel does, in another order).  The 3x3 dynamic kernel stays on the CUDA
// cores in fp32 -- dk is an fp32 quantity and must not be rounded to bf16 -- and is added to the
// accumulators before the single rounding of the result.
//
//   D (16 x-outputs  x  8 rows)  +=  A (16 x 16: Toeplitz block, weights)  x  B (16 x-inputs x 8 rows: image)
//
// The instruction wants, per channel, x-contiguous image rows; NHWC keeps a pixel's channels
// together instead.  A unit's halo tile therefore lands as NHWC (one TMA load, zero fill = the
// padding) in a staging buffer and is transposed into 16 per-channel planes with ldmatrix.trans
// (8 pixels x 8 channels at a time) -- about 5 % of the unit's time -- while the staging buffer is
// already being refilled with the next unit's tile.  Results go back the same way: bf16 into the
// plane, then ldmatrix.trans across the 16 planes with the row addresses chosen so that a lane ends up
// with eight channels of one pixel: one 16-byte store per lane, 32-byte sectors complete.
//
// One CTA per SM, persistent over units (an output tile of 16*NB x 8*NA pixels x 16 channels):
//   warps 0-7   transpose in, then each takes two channels: 13 kernel rows x (NB + 1) input blocks,
//               one ldmatrix.x4 (two row blocks) feeding four MMAs; dynamic 3x3; transpose out.
//   warp 8      tile producer (TMA), warp 9 copy-through of the untouched channels (TMA in / out).
#pragma once
#include "stencil_tma.cuh"

namespace esc { namespace tma { namespace toep {

constexpr int kWarps = 8, kMmaThreads = kWarps * 32, kThreads = kMmaThreads + 64;
constexpr int PT = 16;                              // packed tap pairs per (channel, kernel row): d = -2 .. 13
constexpr int PTAB_BYTES = CG * K13 * PT * 4;       // 13,312

template <int NA_, int NB_>
struct Shape {
    static constexpr int NA = NA_, NB = NB_;         // row blocks of 8, column blocks of 16 per tile
    static constexpr int TH = 8 * NA, TW = 16 * NB;
    static constexpr int ROWS = TH + K13 - 1;        // staged rows
    static constexpr int SW = 16 * (NB + 1);         // staged pixels per row (TW + 12, rounded up to whole input blocks)
    static constexpr int STAGE_BYTES = ROWS * SW * CG * 2;
    // A plane row holds SW bf16 and is padded to 8 * odd elements: the eight 16-byte rows of an ldmatrix
    // then fall in eight different groups of four banks.
    static constexpr int PP = ((SW / 8) | 1) * 8;
    // Plane stride = 4 * odd words (mod 32), for the same reason across planes (transposes read and write
    // the same pixel of eight planes at once).
    static constexpr int PLANE_RAW = ROWS * PP * 2;
    static constexpr int PLANE_BYTES = PLANE_RAW + ((20 - (PLANE_RAW / 4) % 32 + 32) % 32) * 4;
    static_assert(NA % 2 == 0, "row blocks are taken in pairs");
    static_assert(PLANE_BYTES % 16 == 0 && (PLANE_BYTES / 4) % 32 == 20, "plane stride");
    static_assert(STAGE_BYTES % 128 == 0, "staging keeps 128-byte alignment");
};
using Shape64x16 = Shape<2, 4>;

struct Params {
    int B, C, Ca, H, W;
    int tiles_x, tiles_y, groups;
    long long units;
    int copy_cc, copy_cw, copy_cr, slot_stride;
    const __nv_bfloat16* w_large;     // [Ca][13][13]
    const float* dk;                  // [B][Ca][9]
    const float* bias;                // [B][Ca] or nullptr
    __nv_bfloat16* out;
    unsigned* ctrl;
    int wait_first;
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

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kMmaThreads) : "memory"); }
__device__ __forceinline__ float bf16_at(const unsigned char* plane, int row, int col, int pp) {
    const unsigned short v = *reinterpret_cast<const unsigned short*>(plane + ((size_t)row * pp + col) * 2);
    return __uint_as_float((unsigned)v << 16);
}

template <class S, bool kBias>
__global__ void __launch_bounds__(kThreads, 1)
stencil_toeplitz_nhwc_bf16(const __grid_constant__ CUtensorMap map_att, const __grid_constant__ CUtensorMap map_cin,
                           const __grid_constant__ CUtensorMap map_cout, const Params p)
{
    constexpr int NA = S::NA, NB = S::NB, TH = S::TH, TW = S::TW, ROWS = S::ROWS, SW = S::SW, PP = S::PP;
    constexpr int PLANE = S::PLANE_BYTES;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* stage = smem;                                   // NHWC halo tile as it lands: [ROWS][SW][16] bf16
    unsigned char* planes = smem + S::STAGE_BYTES;                 // 16 x [ROWS][PP] bf16
    uint32_t* ptab = reinterpret_cast<uint32_t*>(planes + CG * PLANE);   // [16][13][PT] packed tap pairs
    unsigned char* ring = reinterpret_cast<unsigned char*>(ptab) + PTAB_BYTES;
    u64* bars = reinterpret_cast<u64*>(ring + NSLOT * p.slot_stride);
    const uint32_t full = smem_u32(bars), empty = full + 8, cfull0 = full + 16;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        mbar_init(full, 1);
        mbar_init(empty, kWarps);
        for (int s = 0; s < NSLOT; ++s) mbar_init(cfull0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (p.wait_first) pdl_wait_primary();
    pdl_launch_dependents();

    const long long first = blockIdx.x, stride = gridDim.x;
    const long long my_units = first < p.units ? (p.units - first + stride - 1) / stride : 0;

    if (warp >= kWarps) {
        if (lane != 0) return;
        if (warp == kWarps) {
            // ---- tile producer: the staging buffer is free again once every warp has transposed its share
            bool alive = true;
            for (long long k = 0; k < my_units; ++k) {
                if (k >= 1 && alive) alive = mbar_wait(empty, (unsigned)((k - 1) & 1), p.ctrl, 0xB8000000u);
                const Unit un = decode(first + k * stride, p);
                mbar_expect_tx(full, S::STAGE_BYTES);
                tma_load_4d(smem_u32(stage), &map_att, full, un.g * CG, un.tx * TW - P6, un.ty * TH - P6, un.b);
            }
        } else if (p.copy_cc != 0) {
            // ---- copy-through of the untouched channels (same scheme as the FP32 kernel's copy warp)
            struct Cursor {
                int k, ch, cx0, cy0, cb, col, row; bool live;
                __device__ void enter_unit(const Params& p, int first, int stride) {
                    const Unit un = decode(first + k * stride, p);
                    cx0 = un.tx * S::TW; cy0 = un.ty * S::TH; cb = un.b; col = 0; row = 0; ch = 0;
                    live = un.g == 0;
                }
            };
            const int per_row = TW / p.copy_cw, chunks = per_row * (TH / p.copy_cr);
            const unsigned bytes = (unsigned)(p.copy_cc * p.copy_cw * p.copy_cr * 2);
            const int nunits = (int)my_units, first_i = (int)first, stride_i = (int)stride;
            Cursor ld, st;
            ld.k = st.k = 0;
            if (nunits > 0) { ld.enter_unit(p, first_i, stride_i); st = ld; }
            auto advance = [&](Cursor& c) {
                ++c.ch;
                if (++c.col == per_row) { c.col = 0; ++c.row; }
                if (c.ch == chunks) { ++c.k; if (c.k < nunits) c.enter_unit(p, first_i, stride_i); }
            };
            int issued = 0, stored = 0, lag = 0;
            bool alive = true;
            if (nunits > 0) alive = mbar_wait(full, 0u, p.ctrl, 0xC9000000u);   // the first halo tile goes first
            while (st.k < nunits) {
                if (lag == COPY_DEPTH || ld.k >= nunits) {
                    const int cx = st.cx0 + st.col * p.copy_cw, cy = st.cy0 + st.row * p.copy_cr;
                    if (st.live && cx < p.W && cy < p.H) {
                        const int slot = stored % NSLOT;
                        if (alive) alive = mbar_wait(cfull0 + 8 * slot, (unsigned)((stored / NSLOT) & 1), p.ctrl, 0xC8000000u | (unsigned)slot);
                        tma_store_4d(&map_cout, smem_u32(ring + slot * p.slot_stride), p.Ca, cx, cy, st.cb);
                        bulk_commit();
                        ++stored;
                    }
                    advance(st);
                    --lag;
                }
                if (ld.k < nunits) {
                    const int cx = ld.cx0 + ld.col * p.copy_cw, cy = ld.cy0 + ld.row * p.copy_cr;
                    if (ld.live && cx < p.W && cy < p.H) {
                        const int slot = issued % NSLOT;
                        bulk_wait_read<NSLOT - COPY_DEPTH>();
                        mbar_expect_tx(cfull0 + 8 * slot, bytes);
                        tma_load_4d(smem_u32(ring + slot * p.slot_stride), &map_cin, cfull0 + 8 * slot, p.Ca, cx, cy, ld.cb);
                        ++issued;
                    }
                    advance(ld);
                    ++lag;
                }
            }
            bulk_wait_all<0>();
        }
        return;
    }

    // ======================= the eight working warps ===============================================
    const int g = lane >> 2, t = lane & 3;
    const uint32_t stage_a = smem_u32(stage), planes_a = smem_u32(planes);
    // ldmatrix row addresses: lane l supplies row l & 7 of matrix l >> 3
    const int mi = lane >> 3, mr = lane & 7;
    // indices of this lane's packed tap pairs: P[e], P[e + 8], P[e + 16] with e = 2t - g, clamped into the table
    const int e0 = 2 * t - g;
    const int ia = min(max(e0, -2), 13) + 2, ib = min(max(e0 + 8, -2), 13) + 2, ic = min(max(e0 + 16, -2), 13) + 2;

    int cur_g = -1;
    bool alive = true, dk_ready = p.wait_first != 0;
    for (long long k = 0; k < my_units; ++k) {
        const Unit un = decode(first + k * stride, p);

        // ---- packed tap pairs of this channel group: P[c][i][d + 2] = (LK[c][i][d], LK[c][i][d + 1]), zero outside 0..12
        if (un.g != cur_g) {
            // the last reader of the old table passed the barrier that closed the previous unit
            const unsigned short* wg = reinterpret_cast<const unsigned short*>(p.w_large) + (size_t)un.g * CG * K13 * K13;
            constexpr int N = CG * K13 * PT, PER = N / kMmaThreads;
            static_assert(N % kMmaThreads == 0, "table entries per thread");
            unsigned lo[PER], hi[PER];
#pragma unroll
            for (int u = 0; u < PER; ++u) {                  // all loads in flight together
                const int e = tid + u * kMmaThreads, d = (e % PT) - 2, row = e / PT;   // row = c * 13 + i
                lo[u] = (d >= 0 && d < K13) ? wg[row * K13 + d] : 0u;
                hi[u] = (d + 1 >= 0 && d + 1 < K13) ? wg[row * K13 + d + 1] : 0u;
            }
#pragma unroll
            for (int u = 0; u < PER; ++u) ptab[tid + u * kMmaThreads] = lo[u] | (hi[u] << 16);
            cur_g = un.g;
            // made visible by the barrier after the transposition below
        }

        // ---- the NHWC tile has landed: transpose it into the 16 planes --------------------------------
        if (alive) alive = mbar_wait(full, (unsigned)(k & 1), p.ctrl, 0xA8000000u);
        {
            // a step = 16 pixels of one staged row x 16 channels: four 8x8 matrices (pixel half, channel half)
            constexpr int STEPS = ROWS * (SW / 16);
            const uint32_t src_lane = stage_a + (uint32_t)(((mi >> 1) * 8 + mr) * (CG * 2) + (mi & 1) * 16);
            for (int s = warp; s < STEPS; s += kWarps) {
                const int row = s / (SW / 16), x0 = (s % (SW / 16)) * 16;
                uint32_t r[4];
                ldsm_x4_trans(src_lane + (uint32_t)((row * SW + x0) * (CG * 2)), r);
                // r[j], lane (g, t): channel 8 * (j & 1) + g, pixels x0 + 8 * (j >> 1) + 2t, + 1
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int c = 8 * (j & 1) + g, x = x0 + 8 * (j >> 1) + 2 * t;
                    *reinterpret_cast<uint32_t*>(planes + (size_t)c * PLANE + ((size_t)row * PP + x) * 2) = r[j];
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty);                   // staging may be refilled
        mma_bar();                                           // planes (and the tap table) complete

        // ---- two channels per warp --------------------------------------------------------------------
        // Per channel: 13 kernel rows of tensor-core work into acc, then the dynamic 3x3 kernel on the CUDA
        // cores, fp32 (Eq. 4 line 3, second term), into dacc; dk is waited for after the first channel's
        // tensor-core work of a CTA's first unit, which runs beside the kernel that produces it.
        const unsigned sh = (g & 1) ? 0u : 16u;
        float acc[NB][NA][4], dacc[NB][NA][4];
        float dkv[9];

        auto mma_all = [&](float (&a4)[NB][NA][4], const int c) {
            const uint32_t b_lane = planes_a + (uint32_t)c * PLANE + (uint32_t)((((mi >> 1) * 8 + mr) * PP + (mi & 1) * 8) * 2);
            const uint32_t* pt = ptab + c * (K13 * PT);
#pragma unroll
            for (int q = 0; q < NB; ++q)
#pragma unroll
                for (int r = 0; r < NA; ++r)
#pragma unroll
                    for (int v = 0; v < 4; ++v) a4[q][r][v] = 0.f;
#pragma unroll 1
            for (int i = 0; i < K13; ++i) {
                const uint32_t pa = pt[i * PT + ia], pb = pt[i * PT + ib], pc = pt[i * PT + ic];
                // A0[m][k] = LK[i][k - m] (outputs of block q from inputs of block q),
                // A1[m][k] = LK[i][k - m + 16] (outputs of block q - 1 from inputs of block q)
#pragma unroll
                for (int r2 = 0; r2 < NA / 2; ++r2) {
#pragma unroll
                    for (int q = 0; q <= NB; ++q) {
                        uint32_t b[4];
                        ldsm_x4(b_lane + (uint32_t)(((16 * r2 + i) * PP + 16 * q) * 2), b);
                        if (q < NB) {
                            mma_bf16(a4[q][2 * r2], pa, 0u, pb, pa, b[0], b[1]);
                            mma_bf16(a4[q][2 * r2 + 1], pa, 0u, pb, pa, b[2], b[3]);
                        }
                        if (q >= 1) {
                            mma_bf16(a4[q - 1][2 * r2], pc, pb, 0u, pc, b[0], b[1]);
                            mma_bf16(a4[q - 1][2 * r2 + 1], pc, pb, 0u, pc, b[2], b[3]);
                        }
                    }
                }
            }
        };
        // 3x3 for outputs (x = 16q + 8h + g, y = 8r + 2t) and (x, y + 1): slots [q][r][2h], [2h + 1] (the
        // accumulator layout of the tensor-core instruction).  The three inputs x + 5 .. x + 7 of a plane
        // row sit in two aligned 32-bit words; which halves they are depends on the parity of g alone, so
        // a funnel shift by 0 or 16 lines them up.
        auto dk_all = [&](float (&d4)[NB][NA][4], const int c) {
            const uint32_t* plane32 = reinterpret_cast<const uint32_t*>(planes + (size_t)c * PLANE);
            const float* dp = p.dk + ((size_t)un.b * p.Ca + un.g * CG + c) * 9;
#pragma unroll
            for (int v = 0; v < 9; ++v) dkv[v] = __ldcg(dp + v);
            const float bias = kBias ? __ldg(p.bias + (size_t)un.b * p.Ca + un.g * CG + c) : 0.f;
#pragma unroll
            for (int q = 0; q < NB; ++q)
#pragma unroll
                for (int r = 0; r < NA; ++r)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int wi = (16 * q + 8 * h + g + 5) >> 1, y = 8 * r + 2 * t;
                        float in[4][3];
#pragma unroll
                        for (int a = 0; a < 4; ++a) {
                            const uint32_t w0 = plane32[(y + 5 + a) * (PP / 2) + wi], w1 = plane32[(y + 5 + a) * (PP / 2) + wi + 1];
                            const uint32_t u = __funnelshift_r(w0, w1, sh);
                            in[a][0] = __uint_as_float(u << 16);
                            in[a][1] = __uint_as_float(u & 0xffff0000u);
                            in[a][2] = __uint_as_float((w1 >> sh) << 16);
                        }
                        float s0 = bias, s1 = bias;
#pragma unroll
                        for (int a = 0; a < 3; ++a)
#pragma unroll
                            for (int bcol = 0; bcol < 3; ++bcol) {
                                s0 = fmaf(dkv[a * 3 + bcol], in[a][bcol], s0);
                                s1 = fmaf(dkv[a * 3 + bcol], in[a + 1][bcol], s1);
                            }
                        d4[q][r][2 * h] = s0; d4[q][r][2 * h + 1] = s1;
                    }
        };
        // result of channel c = acc + dacc, rounded once to bf16, into rows 0 .. TH-1, columns 0 .. TW-1 of its plane
        auto write_back = [&](const float (&a4)[NB][NA][4], const float (&d4)[NB][NA][4], const int c) {
            unsigned char* plane = planes + (size_t)c * PLANE;
            __syncwarp();                                    // every lane has read its neighbours
#pragma unroll
            for (int q = 0; q < NB; ++q)
#pragma unroll
                for (int r = 0; r < NA; ++r)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int x = 16 * q + g + 8 * h, y = 8 * r + 2 * t;
                        *reinterpret_cast<__nv_bfloat16*>(plane + ((size_t)y * PP + x) * 2) = __float2bfloat16_rn(a4[q][r][2 * h] + d4[q][r][2 * h]);
                        *reinterpret_cast<__nv_bfloat16*>(plane + ((size_t)(y + 1) * PP + x) * 2) = __float2bfloat16_rn(a4[q][r][2 * h + 1] + d4[q][r][2 * h + 1]);
                    }
        };

#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
            const int c = warp * 2 + cc;
            mma_all(acc, c);
            if (!dk_ready) { pdl_wait_primary(); dk_ready = true; }
            dk_all(dacc, c);
            write_back(acc, dacc, c);
        }
        mma_bar();                                           // all 16 planes hold their results

        // ---- transpose out: 16 pixels x 16 channels per step, one 16-byte store per lane ------------------
        {
            constexpr int STEPS = TH * (TW / 16);
            // The row addresses of an ldmatrix are free: row rho = 2 * tt + e of matrix mi points at plane
            // 8 * (tt & 1) + 2 * mi + e, pixels x0 + 8 * (tt >> 1) .., so that after the transposition lane (g, t)
            // holds, in its four registers, channels 8 * (t & 1) + 0 .. 7 of pixel x0 + 8 * (t >> 1) + g: one
            // 16-byte store, no exchange between lanes.  (Planes c and c + 8 share banks: two wavefronts per matrix.)
            const int tt = mr >> 1, ee = mr & 1;
            const uint32_t src_lane = planes_a + (uint32_t)((8 * (tt & 1) + 2 * mi + ee) * PLANE + (tt >> 1) * 16);
            const int y0 = un.ty * TH, xt0 = un.tx * TW;
            for (int s = warp; s < STEPS; s += kWarps) {
                const int y = s / (TW / 16), x0 = (s % (TW / 16)) * 16;
                uint32_t r[4];
                ldsm_x4_trans(src_lane + (uint32_t)((y * PP + x0) * 2), r);
                const int px = xt0 + x0 + 8 * (t >> 1) + g, py = y0 + y;
                if (px < p.W && py < p.H) {
                    uint4* dst = reinterpret_cast<uint4*>(p.out + (((size_t)un.b * p.H + py) * p.W + px) * p.C + un.g * CG + 8 * (t & 1));
                    *dst = make_uint4(r[0], r[1], r[2], r[3]);
                }
            }
        }
        mma_bar();                                           // the planes are free for the next tile
    }
}

// ---- host side ------------------------------------------------------------------------------
template <class S>
inline long long units_of(int B, int Ca, int H, int W) {
    return (long long)B * (Ca / CG) * ((W + S::TW - 1) / S::TW) * ((H + S::TH - 1) / S::TH);
}

template <class S, bool kBias>
inline int launch_shape(int B, int C, int Ca, int H, int W, const void* x, const void* w_large, const float* dk,
                        const float* bias, void* out, unsigned* ctrl, cudaStream_t st, bool dependent, int* launches,
                        std::string* err) {
    const int cc = C - Ca;
    Params p;
    p.B = B; p.C = C; p.Ca = Ca; p.H = H; p.W = W;
    p.tiles_x = (W + S::TW - 1) / S::TW; p.tiles_y = (H + S::TH - 1) / S::TH; p.groups = Ca / CG;
    p.units = units_of<S>(B, Ca, H, W);
    if (p.units > 0x7fffffffLL) return kNotApplicable;
    p.copy_cc = cc; p.copy_cw = S::TW; p.copy_cr = 1; p.slot_stride = 128;
    if (cc > 0) {
        const int shapes[6][2] = {{S::TW, 4}, {S::TW, 2}, {S::TW, 1}, {S::TW / 2, 1}, {S::TW / 4, 1}, {S::TW / 8, 1}};
        int pick = -1;
        for (int s = 0; s < 6 && pick < 0; ++s)
            if (S::TH % shapes[s][1] == 0 && cc * 2 * shapes[s][0] * shapes[s][1] <= kMaxSlotBytes) pick = s;
        if (pick < 0) return kNotApplicable;
        p.copy_cw = shapes[pick][0]; p.copy_cr = shapes[pick][1];
        p.slot_stride = (cc * 2 * p.copy_cw * p.copy_cr + 127) / 128 * 128;
    }
    p.w_large = static_cast<const __nv_bfloat16*>(w_large);
    p.dk = dk; p.bias = bias; p.out = static_cast<__nv_bfloat16*>(out); p.ctrl = ctrl;
    p.wait_first = dependent ? 0 : 1;

    CUtensorMap m_att, m_cin, m_cout;
    if (!make_map(&m_att, x, B, C, H, W, CG, S::SW, S::ROWS, CU_TENSOR_MAP_L2_PROMOTION_L2_64B)) return kNotApplicable;
    if (cc > 0) {
        if (!make_map(&m_cin, x, B, C, H, W, cc, p.copy_cw, p.copy_cr)) return kNotApplicable;
        if (!make_map(&m_cout, out, B, C, H, W, cc, p.copy_cw, p.copy_cr)) return kNotApplicable;
    } else {
        m_cin = m_att; m_cout = m_att;
    }
    const size_t smem = (size_t)S::STAGE_BYTES + (size_t)CG * S::PLANE_BYTES + PTAB_BYTES + (size_t)NSLOT * p.slot_stride + 64;
    if (smem > 227 * 1024) return kNotApplicable;
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return kNotApplicable;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(stencil_toeplitz_nhwc_bf16<S, kBias>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return kNotApplicable; }
        attr_set[dev] = true;
    }
    const long long grid = p.units < sm_count() ? p.units : sm_count();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, stencil_toeplitz_nhwc_bf16<S, kBias>, m_att, m_cin, m_cout, p);
    if (e != cudaSuccess) {
        char buf[256];
        snprintf(buf, sizeof buf, "stencil_toeplitz_nhwc_bf16 launch: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e));
        *err = buf;
        return 7;  // ESC_ERR_CUDA
    }
    ++*launches;
    return 0;
}

inline bool applies(int C, int Ca, int K, int dtype, int layout) {
    return K == K13 && dtype == 1 /*bf16*/ && layout == kNHWC && Ca % CG == 0 && C % 8 == 0 && C - Ca <= 256;
}

// Launches the tensor-core stencil if the problem fits it: 0 on success, kNotApplicable otherwise, or an ESC_ERR_* code.
inline int try_launch_toeplitz(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x,
                               const void* w_large, const float* dk, const float* bias, void* out, unsigned* ctrl,
                               cudaStream_t st, bool dependent, int* launches, std::string* err, int* tile_w) {
    if (!applies(C, Ca, K, dtype, layout) || sm_count() <= 0) return kNotApplicable;
    *tile_w = Shape64x16::TW;
    return bias ? launch_shape<Shape64x16, true>(B, C, Ca, H, W, x, w_large, dk, bias, out, ctrl, st, dependent, launches, err)
                : launch_shape<Shape64x16, false>(B, C, Ca, H, W, x, w_large, dk, bias, out, ctrl, st, dependent, launches, err);
}

}}}  // namespace esc::tma::toep

// Kernel (b), fast path: TMA-staged, register-tiled fused stencil for K = 13 on NHWC bf16 tensors
// (ESC paper, Section 3.3, Eq. 4 lines 3-4, evaluated in the merged form ZP(dk) + LK^s of Eq. 5).
//
// Work unit: an output tile of one image for one group of 16 attention channels.  The kernel is a
// template over the tile geometry; the description below gives the numbers of the main one (40x40
// tiles, 5x10 outputs per lane), the second one (64x16 tiles, 4x8 outputs per lane) serves maps
// that 40x40 tiles cover or balance badly -- the host picks by a cost estimate.  One CTA per
// SM, persistent over units, three warp groups:
//   warps 0-7  compute.  lane = (patch position q, channel pair p); a warp covers 4 patches of
//              5x10 outputs x 8 channel pairs, two channels at a time with packed fp32 FMAs
//              (fma.rn.f32x2).  The loop runs over the 17 INPUT rows a patch touches: a row is read
//              from shared memory and widened to fp32 once (22 words), then used by up to five
//              output rows, each with its own kernel row (7 broadcast-free 16-byte weight loads).
//              That keeps the non-FMA instructions near 10 % of the issue slots, which matters
//              because a packed FMA takes two issue slots and nothing is issued in its shadow.
//   warp 8     tile producer: one TMA load per unit of the (40+12) x (40+12+1) x 16-channel halo
//              tile into a two-deep ring; coordinates outside the image are zero-filled by the TMA
//              unit, which is the 'same' padding.
//   warp 9     copy-through: streams the untouched channels of the same tile global -> shared ->
//              global with TMA loads and stores through a small ring.
// The helper warps give their registers to the compute warps (setmaxnreg), which need ~200.
// Results are rounded once to bf16, staged in the freed input buffer and written with one TMA
// store per unit (clipped at the image border by the TMA unit).
//
// Shared-memory words of the tile hold one pixel's channel pair (bf16x2); a pixel is 8 words
// (32 bytes), a tile row 53 pixels.  The four patches of a warp form a 2x2 block; with an odd row
// pitch and a patch of 5 rows x 10 columns their first pixels differ mod 4, so the 32 lanes of
// every LDS.32 hit 32 different banks.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <string>
#include <cstdio>
#include <cstdint>

#include "common.cuh"

namespace esc { namespace tma {

constexpr int kNotApplicable = -1;

constexpr int K13 = 13, P6 = 6;
constexpr int CG = 16;                               // channels per unit
constexpr int NPAIR = CG / 2;
static_assert(CG == 16, "index arithmetic below shifts by 4 for the channel group");
constexpr int kComputeWarps = 8;
constexpr int kComputeThreads = kComputeWarps * 32;  // 256
constexpr int kThreads = kComputeThreads + 128;      // + helper warp group (producer, copy, 2 idle)
constexpr int kLaunchRegs = 152;                      // 384*152 = 58,368: leaves 7,168 registers (1,792 per sub-partition) for one GAP block (128 x 56) per SM
constexpr int kComputeRegs = 208, kHelperRegs = 40;   // after reallocation: 256*208 + 128*40 = 58,368
constexpr int WSM_FLOATS = K13 * 7 * NPAIR * 4;      // [i][jj][pair][4]: taps 2jj,2jj+1 of both channels
constexpr int WSM_BYTES = (WSM_FLOATS * 4 + 127) / 128 * 128;
constexpr int LKC_BYTES = (CG * 9 * 4 + 127) / 128 * 128;
constexpr int NSLOT = 2, COPY_DEPTH = 1;             // copy ring: slots, loads in flight (few large chunks: the copy
                                                     // thread shares a scheduler with two compute warps and every
                                                     // instruction it issues delays them, then the whole block at the barriers)
constexpr int kMaxSlotBytes = 16384;
constexpr unsigned kSpinLimit = 1u << 20;    // polls before a wait gives up (each poll may suspend up to the hint):
constexpr unsigned kSuspendHintNs = 1000;    // a wait that never ends gives up after about one second

// Tile geometry.  A lane owns a patch of OY rows x OX columns of outputs; a tile is LXP x LYP
// patches (always 32, i.e. 8 warps of 4 patches x 8 channel pairs).  The 32 lanes of an LDS.32 hit
// 32 different banks when the four patches of a warp start at pixel indices that differ mod 4:
//   kBlock2x2   the four patches form a 2x2 block: needs OX = 2 (mod 4) and an odd OY * PITCH;
//   otherwise   they are stacked vertically: conflict-free only for an odd OY * PITCH.
template <int OX_, int OY_, int LXP_, int LYP_, bool kBlock2x2_>
struct Geom {
    static constexpr int OX = OX_, OY = OY_, LXP = LXP_, LYP = LYP_;
    static constexpr bool kBlock2x2 = kBlock2x2_;
    static constexpr int TW = OX * LXP, TH = OY * LYP;            // outputs per tile
    static constexpr int THP = TH + K13 - 1;                      // staged rows
    static constexpr int PITCH = (TW + K13 - 1) | 1;              // staged pixels per row, odd on purpose
    static constexpr int NW = OX + K13 - 1;                       // input pixels per patch row
    static constexpr int NR = OY + K13 - 1;                       // input rows per patch
    static constexpr int TILE_BYTES = THP * PITCH * CG * 2;
    static constexpr int OUT_TILE_BYTES = TH * TW * CG * 2;       // staged result, reuses the input buffer
    static_assert(LXP * LYP == 4 * kComputeWarps, "one patch per (warp, q)");
    static_assert(TILE_BYTES % 128 == 0, "tile buffers must keep 128-byte alignment");
    static_assert(OUT_TILE_BYTES <= TILE_BYTES, "the result tile is staged in the input buffer");
    static_assert(kBlock2x2 ? ((OY * PITCH) % 2 == 1 && OX % 4 == 2 && LXP % 2 == 0 && LYP % 2 == 0) : (LYP % 4 == 0),
                  "patch-to-lane mapping does not fit the tile");
    __device__ static __forceinline__ void patch_of(int warp, int q, int& lx, int& ly) {
        if (kBlock2x2) {
            lx = 2 * (warp % (LXP / 2)) + (q & 1);
            ly = 2 * (warp / (LXP / 2)) + (q >> 1);
        } else {
            lx = warp % LXP;
            ly = 4 * (warp / LXP) + q;
        }
    }
};
// 40x40 tiles (52 x 53 x 16 staged, 88,192 bytes): the best ratio of arithmetic to halo, loads and
// per-unit overhead; used whenever the tile count balances over the SMs.
using Geom40 = Geom<10, 5, 4, 8, true>;
// 64x16 tiles (28 x 77 x 16 staged, 68,992 bytes) for maps that 40x40 tiles cover badly (a 64x64
// patch: 64 % useful outputs) or that give too few 40x40 tiles to occupy the SMs.  OY = 4 makes the
// four stacked patches of a warp share banks (4-way conflict on the 20 input loads per row):
// measured 15 % more time per FMA than Geom40, 64x20 tiles (OY = 5, conflict-free) 3 % more;
// on 64x64 patches the exact cover still wins (45.7 us against 50.3 and 58.0).
using Geom64 = Geom<8, 4, 8, 4, false>;

struct Params {
    int B, C, Ca, H, W;
    int tiles_x, tiles_y, groups;     // units = B * groups * tiles_y * tiles_x
    long long units;
    int copy_cc, copy_cw, copy_cr;    // copy box: channels, pixels, rows (copy_cc == 0: nothing to copy)
    int slot_stride;                  // bytes between ring slots (multiple of 128)
    const __nv_bfloat16* w_large;     // [Ca][13][13]
    const __nv_bfloat16* w_point;     // [16][16] point-wise filter LK^c of the decomposed form, or nullptr
    const float* dk;                  // [B][Ca][9]
    const float* bias;                // [B][Ca] constant added to every output of (image, channel), or nullptr
    unsigned* ctrl;                   // status words or nullptr
    int wait_first;                   // 1: nothing may be read before the previous kernel of the stream has finished
};

// ---- PTX wrappers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One poll of a phase; the thread is suspended by the hardware until the phase completes or the
// time hint (ns) runs out, so a waiting thread issues almost no instructions.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendHintNs) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls, records where, and lets the caller carry on.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, unsigned parity, unsigned* ctrl, unsigned where) {
    for (unsigned n = 0; n < kSpinLimit; ++n)
        if (mbar_try_wait(bar, parity)) return true;
    if (ctrl) { atomicExch(ctrl, kDevTimeout); atomicExch(ctrl + 1, where); }
    return false;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
        ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void compute_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kComputeThreads) : "memory"); }
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

typedef unsigned long long u64;
__device__ __forceinline__ u64 pack2(float lo, float hi) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ void fma2(u64& d, u64 a, u64 b) { asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b)); }

struct Unit { int b, g, ty, tx; };
__device__ __forceinline__ Unit decode_unit(long long u64v, const Params& p) {
    unsigned u = (unsigned)u64v;                             // the host guarantees units < 2^31
    Unit r;
    r.tx = (int)(u % (unsigned)p.tiles_x); u /= (unsigned)p.tiles_x;
    r.ty = (int)(u % (unsigned)p.tiles_y); u /= (unsigned)p.tiles_y;
    r.g = (int)(u % (unsigned)p.groups);
    r.b = (int)(u / (unsigned)p.groups);
    return r;
}

__device__ __forceinline__ int wsm_index(int c, int i, int j) {
    return ((i * 7 + (j >> 1)) * NPAIR + (c >> 1)) * 4 + (j & 1) * 2 + (c & 1);
}

// D (16x8, fp32) = A (16x16, bf16, row-major) x B (16x8, bf16, column-major): the warp-level tensor-core
// instruction, used only for the small point-wise mix below.
__device__ __forceinline__ void mma_16x8x16_bf16(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// Decomposed form of Eq. 5, first factor: every staged pixel's 16 channels are replaced in place by
// LK^c applied to them, F <- F * LK^c (1x1 convolution, out[n] = sum_k w_point[n][k] in[k]), with fp32
// accumulation on the tensor cores and one rounding back to bf16.  Zero-filled halo pixels stay zero,
// which is the zero padding of the mixed feature map.  A warp takes 16 pixels at a time: pixel rows are
// the A matrix, LK^c the B matrix in two halves of 8 output channels; a lane reads and writes only its
// own eight bytes of two pixels, so the update needs no staging.
// The tensor-core instruction sums over k and fills column n in a fixed lane layout, but which channel
// a k or an n stands for is free as long as A, B and D agree.  Both are permuted here so that lane
// (g, t) -- g = lane / 4, t = lane % 4 -- deals with channels 4t..4t+3 only, on the input and on the
// output side: its A fragment is one 8-byte read per pixel, its D fragments one 8-byte write, and a
// warp's reads and writes cover whole 256-byte runs of the tile (no bank conflicts; with the natural
// order every access touches half of each 32-byte pixel and the mix is twice as slow, bound by
// shared-memory bandwidth either way).
//   k = 2t + e      <-> input channel 4t + e          k = 8 + 2t + e      <-> input channel 4t + 2 + e
//   n = 2j + e, first half <-> output channel 4j + e  second half         <-> output channel 4j + 2 + e
__device__ __forceinline__ void load_mix_fragments(const __nv_bfloat16* __restrict__ w_point, int lane, uint32_t (&bf)[4]) {
    const int g = lane >> 2, t = lane & 3;
    const uint32_t* wp = reinterpret_cast<const uint32_t*>(w_point);        // word n*8 + c/2 = (w[n][c], w[n][c+1])
    const int n0 = 4 * (g >> 1) + (g & 1), n1 = n0 + 2;                      // output channels of column g in either half
    bf[0] = __ldg(wp + n0 * 8 + 2 * t); bf[1] = __ldg(wp + n0 * 8 + 2 * t + 1);
    bf[2] = __ldg(wp + n1 * 8 + 2 * t); bf[3] = __ldg(wp + n1 * 8 + 2 * t + 1);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

template <int NPIX>
__device__ __forceinline__ void pointwise_mix_tile(uint32_t* tile, const uint32_t (&bf)[4], int warp, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const uint32_t b0[2] = {bf[0], bf[1]}, b1[2] = {bf[2], bf[3]};
    uint2* t2 = reinterpret_cast<uint2*>(tile) + t;          // pixel p, channels 4t..4t+3: t2[p * 4]
    constexpr int U = 4, STEP = kComputeWarps * 16;          // groups of 16 pixels in flight per warp
#pragma unroll 1
    for (int base = warp * 16; base < NPIX; base += U * STEP) {
        // all loads, then all products, then all stores: a warp issues in order and the loads of one
        // group may not move above the stores of another (same array)
        uint32_t a[U][4];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int pa = base + u * STEP + g, pb = pa + 8;
            const uint2 va = pa < NPIX ? t2[pa * 4] : make_uint2(0u, 0u);
            const uint2 vb = pb < NPIX ? t2[pb * 4] : make_uint2(0u, 0u);
            a[u][0] = va.x; a[u][2] = va.y; a[u][1] = vb.x; a[u][3] = vb.y;
        }
        float d0[U][4], d1[U][4];
#pragma unroll
        for (int u = 0; u < U; ++u) {
#pragma unroll
            for (int e = 0; e < 4; ++e) d0[u][e] = d1[u][e] = 0.f;
            mma_16x8x16_bf16(d0[u], a[u], b0);
            mma_16x8x16_bf16(d1[u], a[u], b1);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int pa = base + u * STEP + g, pb = pa + 8;
            if (pa < NPIX) t2[pa * 4] = make_uint2(pack_bf16x2(d0[u][0], d0[u][1]), pack_bf16x2(d1[u][0], d1[u][1]));
            if (pb < NPIX) t2[pb * 4] = make_uint2(pack_bf16x2(d0[u][2], d0[u][3]), pack_bf16x2(d1[u][2], d1[u][3]));
        }
    }
}

template <class G, bool kMix, bool kBias>
__global__ void __maxnreg__(kLaunchRegs)
stencil_tma_nhwc_bf16(const __grid_constant__ CUtensorMap map_att, const __grid_constant__ CUtensorMap map_cin,
                      const __grid_constant__ CUtensorMap map_cout, const __grid_constant__ CUtensorMap map_res,
                      const Params p)
{
    // The dynamic shared window starts 1024-byte aligned; indexing it directly (no pointer rounding
    // through integers) lets the compiler keep every access in the shared address space.
    constexpr int OX = G::OX, OY = G::OY, TW = G::TW, TH = G::TH, PITCH = G::PITCH, NW = G::NW;
    constexpr int TILE_BYTES = G::TILE_BYTES;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* tilebuf = smem;                                            // 2 x TILE_BYTES
    float* wsm = reinterpret_cast<float*>(smem + 2 * TILE_BYTES);             // large kernel of the current channel group
    float* lkc = reinterpret_cast<float*>(smem + 2 * TILE_BYTES + WSM_BYTES); // centre 3x3 of LK^s alone
    unsigned char* ring = smem + 2 * TILE_BYTES + WSM_BYTES + LKC_BYTES;      // NSLOT x slot_stride
    u64* bars = reinterpret_cast<u64*>(ring + NSLOT * p.slot_stride);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + 2), cfull0 = smem_u32(bars + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        mbar_init(full0, 1); mbar_init(full0 + 8, 1);
        mbar_init(empty0, 1); mbar_init(empty0 + 8, 1);
        for (int s = 0; s < NSLOT; ++s) mbar_init(cfull0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // Programmatic stream serialization.  As the dependent of the GAP kernel (wait_first == 0) this
    // kernel starts beside it: x is complete (the GAP kernel lets its dependent go only after its own
    // predecessor has finished), dk is waited for where it is needed.  Launched on its own
    // (wait_first == 1) it may be resident before its predecessor has finished and waits here.  Either
    // way the next kernel of the stream may be scheduled from now on; it has to wait for this grid
    // itself before it touches anything, as the two kernels of this library do.
    if (p.wait_first) pdl_wait_primary();
    pdl_launch_dependents();

    const long long first = blockIdx.x, stride = gridDim.x;
    const long long my_units = first < p.units ? (p.units - first + stride - 1) / stride : 0;

    if (warp >= kComputeWarps) {
        // ======================= helper warp group ================================================
        reg_dec<kHelperRegs>();
        if (lane != 0) return;
        if (warp == kComputeWarps) {
            // ---- tile producer: unit k goes to buffer k & 1 once its previous user has released it
            bool alive = true;
            for (long long k = 0; k < my_units; ++k) {
                const int buf = (int)(k & 1);
                if (k >= 2 && alive) alive = mbar_wait(empty0 + 8 * buf, (unsigned)(((k >> 1) - 1) & 1), p.ctrl, 0xB0000000u | (unsigned)buf);
                const Unit un = decode_unit(first + k * stride, p);
                mbar_expect_tx(full0 + 8 * buf, TILE_BYTES);
                tma_load_4d(smem_u32(tilebuf + (size_t)buf * TILE_BYTES), &map_att, full0 + 8 * buf,
                            un.g * CG, un.tx * TW - P6, un.ty * TH - P6, un.b);
            }
        } else if (warp == kComputeWarps + 1 && p.copy_cc != 0) {
            // ---- copy-through of the untouched channels: TMA in, TMA out ---------------------------
            // Two cursors walk the CTA's chunk stream (units in order, chunks row-major inside a
            // unit): the load cursor runs COPY_DEPTH chunks ahead of the store cursor.  No division
            // in the loop: this thread competes with FMA-bound warps for issue slots.
            struct Cursor {
                int k, ch, cx0, cy0, cb, col, row; bool live;
                __device__ void enter_unit(const Params& p, int first, int stride) {
                    const Unit un = decode_unit(first + k * stride, p);
                    cx0 = un.tx * G::TW; cy0 = un.ty * G::TH; cb = un.b; col = 0; row = 0; ch = 0;
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
            // The copy has the whole kernel to finish, the compute warps cannot start without the
            // first halo tile: let that tile land before competing with it for DRAM.
            if (nunits > 0) alive = mbar_wait(full0, 0u, p.ctrl, 0xC1000000u);
            while (st.k < nunits) {
                // store the oldest chunk once COPY_DEPTH loads are in flight (or nothing is left to load)
                if (lag == COPY_DEPTH || ld.k >= nunits) {
                    const int cx = st.cx0 + st.col * p.copy_cw, cy = st.cy0 + st.row * p.copy_cr;
                    if (st.live && cx < p.W && cy < p.H) {
                        const int slot = stored % NSLOT;
                        if (alive) alive = mbar_wait(cfull0 + 8 * slot, (unsigned)((stored / NSLOT) & 1), p.ctrl, 0xC0000000u | (unsigned)slot);
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
                        // the store that last used this slot is at least NSLOT - COPY_DEPTH + 1 groups back
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

    // ======================= compute warps ========================================================
    reg_inc<kComputeRegs>();
    const int q = lane >> 3, pr = lane & 7;                 // which of the warp's four patches, channel pair
    int lx, ly;
    G::patch_of(warp, q, lx, ly);
    const int lane_word = ((ly * OY) * PITCH + lx * OX) * NPAIR + pr;

    int cur_g = -1, merged_b = -1;
    bool alive = true, dk_ready = p.wait_first != 0;
    for (long long k = 0; k < my_units; ++k) {
        const Unit un = decode_unit(first + k * stride, p);
        const int buf = (int)(k & 1);

        // ---- large-kernel taps of this channel group -> shared, fp32, pair-interleaved ----------
        if (un.g != cur_g) {
            if (cur_g >= 0) compute_bar();                  // everyone is done with the old table
            const __nv_bfloat16* wg = p.w_large + (size_t)un.g * CG * K13 * K13;
            // Element e = 16 * tap + channel: the 16 lanes that share a tap write the 16 words of one
            // (i, jj, j & 1) group -- no bank conflicts in the scatter, one division per element.
            constexpr int N = CG * K13 * K13, PER = (N + kComputeThreads - 1) / kComputeThreads;
            float v[PER];
#pragma unroll
            for (int t = 0; t < PER; ++t) {                 // all loads in flight together
                const int e = tid + t * kComputeThreads;
                v[t] = e < N ? __bfloat162float(wg[(e & (CG - 1)) * (K13 * K13) + (e >> 4)]) : 0.f;
            }
#pragma unroll
            for (int t = 0; t < PER; ++t) {
                const int e = tid + t * kComputeThreads;
                if (e < N) {
                    const int c = e & (CG - 1), tap = e >> 4;
                    const int i = tap / K13, j = tap - i * K13;
                    wsm[wsm_index(c, i, j)] = v[t];
                    if (i >= 5 && i <= 7 && j >= 5 && j <= 7) lkc[c * 9 + (i - 5) * 3 + (j - 5)] = v[t];
                }
            }
            if (tid < CG * K13) wsm[wsm_index(tid / K13, tid % K13, K13)] = 0.f;   // pad tap 13
            cur_g = un.g; merged_b = -1;
            compute_bar();
        }

        uint32_t mixb[4];
        if (kMix) load_mix_fragments(p.w_point, lane, mixb);   // issued before the wait: a cold miss hides behind the tile

        if (alive) alive = mbar_wait(full0 + 8 * buf, (unsigned)((k >> 1) & 1), p.ctrl, 0xA0000000u | (unsigned)buf);

        u64 acc[OY][OX];
        if (kBias) {                                         // the backward pass adds a constant per (image, channel)
            const u64 z = pack2(__ldg(p.bias + (size_t)un.b * p.Ca + un.g * CG + 2 * pr),
                                __ldg(p.bias + (size_t)un.b * p.Ca + un.g * CG + 2 * pr + 1));
#pragma unroll
            for (int a = 0; a < OY; ++a)
#pragma unroll
                for (int c = 0; c < OX; ++c) acc[a][c] = z;
        } else {
#pragma unroll
            for (int a = 0; a < OY; ++a)
#pragma unroll
                for (int c = 0; c < OX; ++c) acc[a][c] = 0ull;
        }

        unsigned char* tbuf = tilebuf + (size_t)buf * TILE_BYTES;
        if (kMix) {                                          // Eq. 5: the depth-wise stage sees F_att * LK^c
            pointwise_mix_tile<G::THP * G::PITCH>(reinterpret_cast<uint32_t*>(tbuf), mixb, warp, lane);
            compute_bar();
        }
        const uint32_t* tw = reinterpret_cast<const uint32_t*>(tbuf) + lane_word;
        const float4* wlane = reinterpret_cast<const float4*>(wsm) + pr;

        // One input row r of the patch window: read once, widened once, applied to every output row
        // it belongs to.
        auto do_row = [&](const int r) {
            // input row r of the patch window: read once, widen to fp32 pairs once
            u64 in[NW];
            const uint32_t* rn = tw + r * (PITCH * NPAIR);
#pragma unroll
            for (int kk = 0; kk < NW; ++kk) {
                const uint32_t v = rn[kk * NPAIR];
                in[kk] = pack2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
            }
#pragma unroll
            for (int oy = 0; oy < OY; ++oy) {
                const int i = r - oy;                       // kernel row that maps input row r to output row oy
                if (i >= 0 && i < K13) {                    // same for the whole warp
                    u64 w[K13];
                    const float4* wr = wlane + i * (7 * NPAIR);
#pragma unroll
                    for (int jj = 0; jj < 7; ++jj) {
                        const float4 v = wr[jj * NPAIR];
                        w[2 * jj] = pack2(v.x, v.y);
                        if (2 * jj + 1 < K13) w[2 * jj + 1] = pack2(v.z, v.w);
                    }
#pragma unroll
                    for (int kk = 0; kk < NW; ++kk) {
#pragma unroll
                        for (int j = 0; j < K13; ++j) {
                            const int ox = kk - j;
                            if (ox >= 0 && ox < OX) fma2(acc[oy][ox], w[j], in[kk]);
                        }
                    }
                }
            }
        };

        // Input rows 0-4 and 12-16 only meet kernel rows 0-4 and 8-12; rows 5-11 also meet kernel rows
        // 5-7, whose centre holds the dynamic taps.  Taking them last means the kernel that produces dk
        // is needed only when about half of the first unit is done, so the two kernels run side by
        // side.  Two plain loops (rather than one loop with a special step) keep each loop body free of
        // the barrier code: measured 8 % faster.
#pragma unroll 1
        for (int step = 0; step < 2 * OY; ++step) do_row(step < OY ? step : step + (K13 - 1) - OY);
        if (merged_b != un.b) {
            if (!dk_ready) { pdl_wait_primary(); dk_ready = true; }
            float dkv = 0.f;                                 // fetched before the barrier so its latency hides behind the stragglers
            if (tid < CG * 9) dkv = __ldcg(p.dk + ((size_t)un.b * p.Ca + un.g * CG + tid / 9) * 9 + tid % 9);
            compute_bar();                                   // nobody still reads the old centre taps
            if (tid < CG * 9) {                              // rows 5-7, columns 5-7: LK^s + dk  (Eq. 5)
                const int c = tid / 9, tap = tid % 9;
                wsm[wsm_index(c, 5 + tap / 3, 5 + tap % 3)] = lkc[tid] + dkv;
            }
            merged_b = un.b;
            compute_bar();
        }
#pragma unroll 1
        for (int r = OY; r < K13 - 1; ++r) do_row(r);

        // ---- epilogue: round once to bf16, stage the TH x TW x 16 result in the freed input buffer,
        //      one TMA store (the TMA unit clips at the image border) ---------------------------
        compute_bar();                                       // every warp has finished reading this buffer
        {
            uint32_t* sw = reinterpret_cast<uint32_t*>(tbuf) + ((ly * OY) * TW + lx * OX) * NPAIR + pr;
#pragma unroll
            for (int oy = 0; oy < OY; ++oy)
#pragma unroll
                for (int ox = 0; ox < OX; ++ox) {
                    float lo, hi;
                    unpack2(acc[oy][ox], lo, hi);
                    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
                    sw[(oy * TW + ox) * NPAIR] = *reinterpret_cast<const uint32_t*>(&h);
                }
        }
        fence_async_smem();
        compute_bar();
        if (tid == 0) {
            tma_store_4d(&map_res, smem_u32(tbuf), un.g * CG, un.tx * TW, un.ty * TH, un.b);
            bulk_commit();
            bulk_wait_read<0>();                             // the buffer may be refilled now
            mbar_arrive(empty0 + 8 * buf);
        }
    }
    if (tid == 0) bulk_wait_all<0>();
}

// ---- host side ------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(sym);
    }();
    return fn;
}

// bf16 NHWC tensor [B][H][W][C] as a 4-D map {C, W, H, B} with the given box.
inline bool make_map(CUtensorMap* m, const void* base, int B, int C, int H, int W, int bc, int bw, int bh,
                     CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_128B) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    const cuuint32_t box[4] = {(cuuint32_t)bc, (cuuint32_t)bw, (cuuint32_t)bh, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, promo,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kMaxDevices = 64;

// Index of the current device, or -1.
inline int current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

// SM count of the current device (asked once per device).
inline int sm_count() {
    static int cached[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return 0;
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev] = v;
    }
    return cached[dev];
}

// Units of one launch with geometry G, and the same count as waves over the SMs.
template <class G>
inline long long units_of(int B, int Ca, int H, int W) {
    return (long long)B * (Ca / CG) * ((W + G::TW - 1) / G::TW) * ((H + G::TH - 1) / G::TH);
}
// Relative cost of a launch: every CTA walks ceil(units / SMs) units, each costing its tile area
// plus a fixed per-unit overhead (table merge, barriers, epilogue: about 200 pixels' worth of
// arithmetic); per_fma is the geometry's cost per FMA relative to the 40x40 tile.
template <class G>
inline double cost_of(int B, int Ca, int H, int W, int sms, double per_fma) {
    const long long u = units_of<G>(B, Ca, H, W);
    const long long waves = (u + sms - 1) / sms;
    return (double)waves * ((double)G::TW * G::TH * per_fma + 200.0);
}

template <class G, bool kMix, bool kBias>
inline int launch_geom(int B, int C, int Ca, int H, int W, const void* x, const void* w_large, const void* w_point,
                       const float* dk, const float* bias, void* out, unsigned* ctrl, cudaStream_t st, bool dependent,
                       int* launches, std::string* err) {
    const int cc = C - Ca;
    Params p;
    p.B = B; p.C = C; p.Ca = Ca; p.H = H; p.W = W;
    p.tiles_x = (W + G::TW - 1) / G::TW; p.tiles_y = (H + G::TH - 1) / G::TH; p.groups = Ca / CG;
    p.units = units_of<G>(B, Ca, H, W);
    if (p.units > 0x7fffffffLL) return kNotApplicable;
    p.copy_cc = cc; p.copy_cw = G::TW; p.copy_cr = 1; p.slot_stride = 128;
    if (cc > 0) {
        // chunk = copy_cw pixels x copy_cr rows of the tile; both divide the tile
        static_assert(G::TH % 4 == 0 && G::TW % 8 == 0, "copy chunk shapes");
        const int shapes[6][2] = {{G::TW, 4}, {G::TW, 2}, {G::TW, 1}, {G::TW / 2, 1}, {G::TW / 4, 1}, {G::TW / 8, 1}};
        int pick = -1;
        for (int s = 0; s < 6 && pick < 0; ++s)
            if (cc * 2 * shapes[s][0] * shapes[s][1] <= kMaxSlotBytes) pick = s;
        if (pick < 0) return kNotApplicable;
        p.copy_cw = shapes[pick][0]; p.copy_cr = shapes[pick][1];
        p.slot_stride = (cc * 2 * p.copy_cw * p.copy_cr + 127) / 128 * 128;
    }
    p.w_large = static_cast<const __nv_bfloat16*>(w_large);
    p.w_point = static_cast<const __nv_bfloat16*>(w_point);
    p.dk = dk;
    p.bias = bias;
    p.ctrl = ctrl;
    p.wait_first = dependent ? 0 : 1;

    CUtensorMap m_att, m_cin, m_cout, m_res;
    // The halo tile gates the start of the arithmetic: fetch no more than its own 32-byte sectors need
    // (64-byte promotion measured fastest; 128-byte promotion drags the copy-through channels along).
    if (!make_map(&m_att, x, B, C, H, W, CG, G::PITCH, G::THP, CU_TENSOR_MAP_L2_PROMOTION_L2_64B)) return kNotApplicable;
    if (!make_map(&m_res, out, B, C, H, W, CG, G::TW, G::TH)) return kNotApplicable;
    if (cc > 0) {
        if (!make_map(&m_cin, x, B, C, H, W, cc, p.copy_cw, p.copy_cr)) return kNotApplicable;
        if (!make_map(&m_cout, out, B, C, H, W, cc, p.copy_cw, p.copy_cr)) return kNotApplicable;
    } else {
        m_cin = m_att; m_cout = m_att;
    }

    const size_t smem = 2 * (size_t)G::TILE_BYTES + WSM_BYTES + LKC_BYTES + (size_t)NSLOT * p.slot_stride + 128;
    static bool attr_set[kMaxDevices] = {};                  // function attributes are per device; one array per instantiation
    const int dev = current_device();
    if (dev < 0) return kNotApplicable;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(stencil_tma_nhwc_bf16<G, kMix, kBias>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return kNotApplicable; }
        attr_set[dev] = true;
    }
    if (smem > 227 * 1024) return kNotApplicable;

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
    cudaError_t e = cudaLaunchKernelEx(&cfg, stencil_tma_nhwc_bf16<G, kMix, kBias>, m_att, m_cin, m_cout, m_res, p);
    if (e != cudaSuccess) {
        char buf[256];
        snprintf(buf, sizeof buf, "stencil_tma_nhwc_bf16 launch: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e));
        *err = buf;
        return 7;  // ESC_ERR_CUDA
    }
    ++*launches;
    return 0;
}

// Launches the fast kernel if the problem fits it.  Returns 0 on success, kNotApplicable if the
// generic kernel has to run instead, or an ESC_ERR_* code.  *tile_w: in, the tile width asked
// for (0 = choose by cost); out, the one used.
inline int try_launch(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x,
                      const void* w_large, const void* w_point, const float* dk, const float* bias, void* out,
                      unsigned* ctrl, cudaStream_t st, bool dependent, int* launches, std::string* err, int* tile_w) {
    if (K != K13 || dtype != 1 /*bf16*/ || layout != kNHWC) return kNotApplicable;
    if (Ca % CG != 0 || C % 8 != 0) return kNotApplicable;
    if (C - Ca > 256) return kNotApplicable;
    if (w_point && Ca != CG) return kNotApplicable;         // the mix needs all C_a channels of a pixel in one tile
    if (w_point && (reinterpret_cast<uintptr_t>(w_point) & 3) != 0) return kNotApplicable;   // read as 32-bit words
    const int sms = sm_count();
    if (sms <= 0) return kNotApplicable;
    const bool use64 = *tile_w == Geom64::TW ||
                       (*tile_w != Geom40::TW && cost_of<Geom64>(B, Ca, H, W, sms, 1.15) < cost_of<Geom40>(B, Ca, H, W, sms, 1.0));
    // the combinations in use: plain, with the point-wise mix, with the backward pass's constants
#define ESC_TMA_ARGS B, C, Ca, H, W, x, w_large, w_point, dk, bias, out, ctrl, st, dependent, launches, err
    if (w_point && bias) return kNotApplicable;
    if (use64) {
        *tile_w = Geom64::TW;
        return w_point ? launch_geom<Geom64, true, false>(ESC_TMA_ARGS)
             : bias    ? launch_geom<Geom64, false, true>(ESC_TMA_ARGS)
                       : launch_geom<Geom64, false, false>(ESC_TMA_ARGS);
    }
    *tile_w = Geom40::TW;
    return w_point ? launch_geom<Geom40, true, false>(ESC_TMA_ARGS)
         : bias    ? launch_geom<Geom40, false, true>(ESC_TMA_ARGS)
                   : launch_geom<Geom40, false, false>(ESC_TMA_ARGS);
#undef ESC_TMA_ARGS
}

}}  // namespace esc::tma

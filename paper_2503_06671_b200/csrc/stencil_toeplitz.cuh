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
#include "gap_dynkernel.cuh"

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
    static constexpr int BOX_BYTES = TH * TW * CG * 2;   // a tile's interior alone
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
    const __nv_bfloat16* w_point;     // kMix: [16][16] point-wise filter LK^c of the decomposed form (Eq. 5), row = output channel
    const float* dk;                  // [B][Ca][9]
    const float* bias;                // [B][Ca] or nullptr
    __nv_bfloat16* out;
    unsigned* ctrl;
    int wait_first;
    // Fused stage 1 (kFused): the estimator's weights (bf16; one layer when hidden == 0, see gap_dynkernel.cuh),
    // one slot of 16 partial sums per unit, and per image an arrival counter and a flag that counts launches.
    const __nv_bfloat16 *w_last, *b_last, *w_down, *b_down;
    int hidden;
    float* gpart;
    unsigned *garr, *gflag;
    int upi;                          // units per image = groups * tiles_y * tiles_x
};
constexpr int kFusedMaxCa = 128;      // channels the fused estimator keeps in shared memory
// scratch of the fused stage 1, a multiple of 128 bytes (the copy ring behind it is a TMA destination)
constexpr int FUSED_SMEM_FLOATS = (kMmaThreads + kFusedMaxCa + kMaxHidden + CG * 9 + 2 * kWarps * CG + 31) / 32 * 32;
constexpr int kMaxFusedUnits = 8;     // units a CTA may walk in the one-launch form (kMany: more than two)
constexpr unsigned kFlagPolls = 1u << 22;   // polls of another CTA's flag before a wait gives up (about half a second)

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

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(unsigned* p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// kFused: stage 1 of the module (Eq. 4 line 2) inside this kernel, for launches in which no CTA has more
// than two units.  The pooled means come from the staged tiles themselves: every CTA adds up the interiors
// of its own tiles, which partition the image, writes 16 sums per unit and arrives on the image's counter
// (the atomic is issued by the otherwise idle producer lane, so its round trip stays off the working warps'
// path); the CTA that arrives last advances the image's flag; every CTA then adds the partial sums of the
// image in a fixed order and evaluates the estimator for the 16 channels it is working on.  No second
// kernel, no second pass over the attention channels, and dk is there when the tensor-core work of a CTA's
// first unit is done.  CTAs wait on one another: the launch is cooperative (all CTAs resident, one per SM)
// and every wait is bounded.
// kMix: the decomposed large kernel of Eq. 5 -- the staged tile's 16 attention channels are replaced, pixel by pixel
// and in place, by LK^c applied to them (tensor cores, one rounding to bf16) before the tile is transposed; the pooled
// means of stage 1 are taken from the unmixed tile.
// kMany: the one-launch form for CTAs that walk three to kMaxFusedUnits units.  The interiors of all later units pass,
// half a tile at a time, through the two halves of the buffer that otherwise holds the second unit's interior, and are
// added up before the first unit's products, so that every image's flag advances early; the attention channels (a few
// tens of MB at most) are then in L2 for the tiles' loads.
template <class S, bool kBias, bool kFused, bool kMix = false, bool kMany = false>
__global__ void __launch_bounds__(kThreads, 1)
stencil_toeplitz_nhwc_bf16(const __grid_constant__ CUtensorMap map_att, const __grid_constant__ CUtensorMap map_cin,
                           const __grid_constant__ CUtensorMap map_cout, const __grid_constant__ CUtensorMap map_box,
                           const Params p)
{
    constexpr int NA = S::NA, NB = S::NB, TH = S::TH, TW = S::TW, ROWS = S::ROWS, SW = S::SW, PP = S::PP;
    constexpr int PLANE = S::PLANE_BYTES;
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* stage = smem;                                   // NHWC halo tile as it lands: [ROWS][SW][16] bf16
    unsigned char* planes = smem + S::STAGE_BYTES;                 // 16 x [ROWS][PP] bf16
    uint32_t* ptab = reinterpret_cast<uint32_t*>(planes + CG * PLANE);   // [16][13][PT] packed tap pairs
    float* fsm = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(ptab) + PTAB_BYTES);   // fused stage 1 scratch
    unsigned char* sumbuf = reinterpret_cast<unsigned char*>(fsm) + FUSED_SMEM_FLOATS * 4;       // fused: interior of the second unit's tile
    unsigned char* ring = reinterpret_cast<unsigned char*>(fsm) + (kFused ? FUSED_SMEM_FLOATS * 4 + S::BOX_BYTES : 0);
    u64* bars = reinterpret_cast<u64*>(ring + NSLOT * p.slot_stride);
    const uint32_t full = smem_u32(bars), empty = full + 8, cfull0 = full + 16, sumdone = cfull0 + 8 * NSLOT, boxfull = sumdone + 8,
                   boxfull1 = boxfull + 8, boxfree0 = boxfull1 + 8,     // kMany: two half-tile slots, full and free
                   sumdone_more = boxfree0 + 16;                         // units 1 .. 7: one barrier per unit, each used once
    // (a barrier per unit, not the phases of one: the producer lane may fall several units behind the working warps,
    //  and a wait on a phase's parity is only meaningful one phase back)
    auto sumdone_of = [&](int k) -> uint32_t { return k == 0 ? sumdone : sumdone_more + 8 * (uint32_t)(k - 1); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        mbar_init(full, 1);
        mbar_init(empty, kWarps);
        for (int s = 0; s < NSLOT; ++s) mbar_init(cfull0 + 8 * s, 1);
        mbar_init(sumdone, CG);
        mbar_init(boxfull, 1);
        if (kMany) { mbar_init(boxfull1, 1); mbar_init(boxfree0, 1); mbar_init(boxfree0 + 8, 1); }
        if (kFused)
            for (int k = 1; k < (kMany ? kMaxFusedUnits : 2); ++k) mbar_init(sumdone_of(k), CG);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (p.wait_first) pdl_wait_primary();
    pdl_launch_dependents();

    const long long first = blockIdx.x, stride = gridDim.x;
    const long long my_units = first < p.units ? (p.units - first + stride - 1) / stride : 0;

    if (warp >= kWarps) {
        if (lane != 0) return;
        if (warp == kWarps && kFused && kMany) {
            // ---- stage 1 fused, three or more units: the first unit's halo tile, then the later units' interiors half a
            //      tile at a time through two slots, then the arrivals on the images' counters
            bool alive = true;
            const int n = (int)my_units;
            const Unit u0 = decode(first, p);
            mbar_expect_tx(full, S::STAGE_BYTES);
            tma_load_4d(smem_u32(stage), &map_att, full, u0.g * CG, u0.tx * TW - P6, u0.ty * TH - P6, u0.b);
            unsigned seen[kMaxFusedUnits];
            for (int k = 0; k < n; ++k) seen[k] = ld_acquire(p.gflag + decode(first + k * stride, p).b);
            for (int h = 0; h < 2 * (n - 1); ++h) {
                const int slot = h & 1;
                const Unit un = decode(first + (1 + (h >> 1)) * stride, p);
                if (h >= 2 && alive) alive = mbar_wait(boxfree0 + 8 * slot, (unsigned)(((h >> 1) - 1) & 1), p.ctrl, 0xBA000000u);
                mbar_expect_tx(boxfull + 8 * slot, S::BOX_BYTES / 2);
                tma_load_4d(smem_u32(sumbuf + slot * (S::BOX_BYTES / 2)), &map_box, boxfull + 8 * slot, un.g * CG, un.tx * TW,
                            un.ty * TH + slot * (TH / 2), un.b);
            }
            for (int k = 0; k < n; ++k) {
                const Unit un = decode(first + k * stride, p);
                if (alive) alive = mbar_wait(sumdone_of(k), 0u, p.ctrl, 0xB9000000u | (unsigned)k);
                unsigned old;
                asm volatile("atom.acq_rel.gpu.global.inc.u32 %0, [%1], %2;" : "=r"(old) : "l"(p.garr + un.b), "r"((unsigned)(p.upi - 1)) : "memory");
                if (old == (unsigned)(p.upi - 1)) st_release(p.gflag + un.b, seen[k] + 1u);
            }
            return;
        }
        if (warp == kWarps && kFused) {
            // ---- stage 1 fused: this lane starts the loads -- the first unit's halo tile and, for its sum alone, the
            //      interior of the second unit's tile -- and performs the arrivals on the images' counters once the
            //      working warps have written a unit's 16 sums (the atomic's round trip stays off their path).  The
            //      second unit's halo tile is requested by the working warps when they have transposed the first.
            bool alive = true;
            const Unit u0 = decode(first, p), u1 = decode(first + (my_units > 1 ? stride : 0), p);
            mbar_expect_tx(full, S::STAGE_BYTES);
            tma_load_4d(smem_u32(stage), &map_att, full, u0.g * CG, u0.tx * TW - P6, u0.ty * TH - P6, u0.b);
            if (my_units > 1) {
                mbar_expect_tx(boxfull, S::BOX_BYTES);
                tma_load_4d(smem_u32(sumbuf), &map_box, boxfull, u1.g * CG, u1.tx * TW, u1.ty * TH, u1.b);
            }
            // the flags as they stand before this CTA arrives anywhere: they cannot have advanced yet
            const unsigned seen[2] = {ld_acquire(p.gflag + u0.b), ld_acquire(p.gflag + u1.b)};
            for (int k = 0; k < (int)my_units; ++k) {
                const Unit& un = k == 0 ? u0 : u1;
                if (alive) alive = mbar_wait(sumdone_of(k), 0u, p.ctrl, 0xB9000000u | (unsigned)k);
                // release: the 16 sums (seen through the barrier) are visible to whoever reads the counter or the flag
                unsigned old;
                asm volatile("atom.acq_rel.gpu.global.inc.u32 %0, [%1], %2;" : "=r"(old) : "l"(p.garr + un.b), "r"((unsigned)(p.upi - 1)) : "memory");
                if (old == (unsigned)(p.upi - 1)) st_release(p.gflag + un.b, seen[k] + 1u);   // the counter has wrapped back to 0
            }
            return;
        }
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

    // ---- fused stage 1 ------------------------------------------------------------------------------
    float* f_sub = fsm;                                      // [256] sub-sums of the partial sums
    float* f_mean = fsm + kMmaThreads;                       // [Ca] pooled means of the current image
    float* f_act = f_mean + kFusedMaxCa;                     // [hidden] activations of the two-layer estimator
    float* f_dk = f_act + kMaxHidden;                        // [16][9] dynamic taps of the current (image, group)
    float* f_red = f_dk + CG * 9;                            // [2][8 warps][16] tile sums: consecutive sums alternate between the two
    unsigned flag0[kMany ? kMaxFusedUnits : 2] = {};         // the images' flags as they stood before this launch
    int dk_b = -1, dk_g = -1;
    if (kFused) {
        // read before this CTA arrives anywhere: the flag cannot have advanced yet
        for (int k = 0; k < (int)my_units && k < (kMany ? kMaxFusedUnits : 2); ++k) flag0[k] = ld_acquire(p.gflag + decode(first + k * stride, p).b);
    }
    // Sum of the staged tile's interior per channel (the tiles' interiors partition the image; pixels outside
    // it are zero-filled), in a fixed order; 16 sums to the unit's slot, then the producer lane is told.
    auto tile_sum = [&](const long long unit_index, const unsigned char* src, const int pitch, const int origin, float* const fr, const int k_of_cta) {
        const int gsub = lane >> 3, pr = lane & 7;           // pixel 4i + gsub of a row, channel pair pr: conflict-free
        const uint32_t* st32 = reinterpret_cast<const uint32_t*>(src) + origin * NPAIR;
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int rr = 0; rr < NA; ++rr)
#pragma unroll
            for (int i = 0; i < TW / 4; ++i) {
                const uint32_t v = st32[((warp * NA + rr) * pitch + 4 * i + gsub) * NPAIR + pr];
                s0 += __uint_as_float(v << 16);
                s1 += __uint_as_float(v & 0xffff0000u);
            }
        s0 += __shfl_xor_sync(0xffffffffu, s0, 8);  s1 += __shfl_xor_sync(0xffffffffu, s1, 8);
        s0 += __shfl_xor_sync(0xffffffffu, s0, 16); s1 += __shfl_xor_sync(0xffffffffu, s1, 16);
        if (lane < 8) { fr[warp * CG + 2 * lane] = s0; fr[warp * CG + 2 * lane + 1] = s1; }
        mma_bar();
        if (tid < CG) {
            float tsum = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) tsum += fr[w * CG + tid];
            p.gpart[unit_index * CG + tid] = tsum;
            mbar_arrive(sumdone_of(k_of_cta));
        }
    };
    // dk of (image, group) of `un` into f_dk: wait for the image's flag, add the image's partial sums in a fixed
    // order, evaluate the estimator (Eq. 4 line 2) for the 16 channels of the group.
    auto obtain_dk = [&](const Unit& un, const unsigned seen) {
        if (un.b == dk_b && un.g == dk_g) return;
        if (un.b != dk_b) {
            if (tid == 0 && alive) {
                unsigned n = 0;
                while (ld_acquire(p.gflag + un.b) == seen) {
                    __nanosleep(100);
                    if (++n > kFlagPolls) { if (p.ctrl) { atomicExch(p.ctrl, kDevTimeout); atomicExch(p.ctrl + 1, 0xF0000000u | (unsigned)un.b); } break; }
                }
            }
            mma_bar();
            // means: thread (sub, c) adds tiles sub, sub + nsub, ... of channel c's group; then the sub-sums in order
            const int Ca = p.Ca, nsub = kMmaThreads / Ca, tpi = p.upi / p.groups;
            const int c = tid % Ca, sub = tid / Ca;
            if (sub < nsub) {
                const float* src = p.gpart + ((size_t)un.b * p.upi + (size_t)(c / CG) * tpi) * CG + (c % CG);
                float tsum = 0.f;
                for (int tl = sub; tl < tpi; tl += 16 * nsub) {        // sixteen independent loads, added in order
                    float v[16];
#pragma unroll
                    for (int u = 0; u < 16; ++u) v[u] = tl + u * nsub < tpi ? __ldcg(src + (size_t)(tl + u * nsub) * CG) : 0.f;
#pragma unroll
                    for (int u = 0; u < 16; ++u) tsum += v[u];
                }
                f_sub[tid] = tsum;
            }
            mma_bar();
            if (tid < Ca) {
                float tsum = 0.f;
                for (int j = 0; j < nsub; ++j) tsum += f_sub[j * Ca + tid];
                f_mean[tid] = tsum * (1.0f / (float)((long long)p.H * p.W));
            }
            mma_bar();
            if (p.hidden > 0) {
                for (int j = tid; j < p.hidden; j += kMmaThreads) {
                    float tsum = __bfloat162float(p.b_down[j]);
                    const __nv_bfloat16* wr = p.w_down + (size_t)j * Ca;
                    for (int cc = 0; cc < Ca; ++cc) tsum = fmaf(__bfloat162float(wr[cc]), f_mean[cc], tsum);
                    f_act[j] = gelu_exact(tsum);
                }
                mma_bar();
            }
            dk_b = un.b;
        }
        {
            const float* vin = p.hidden > 0 ? f_act : f_mean;
            const int n_in = p.hidden > 0 ? p.hidden : p.Ca;
            if (tid < CG * 9) {
                const int o = un.g * CG * 9 + tid;
                float a = __bfloat162float(p.b_last[o]);
                const __nv_bfloat16* wr = p.w_last + (size_t)o * n_in;
                for (int c0 = 0; c0 < n_in; c0 += 16) {      // sixteen independent loads, FMAs in input order
                    float wv[16];
#pragma unroll
                    for (int u = 0; u < 16; ++u) wv[u] = c0 + u < n_in ? __bfloat162float(wr[c0 + u]) : 0.f;
#pragma unroll
                    for (int u = 0; u < 16; ++u)
                        if (c0 + u < n_in) a = fmaf(wv[u], vin[c0 + u], a);
                }
                f_dk[tid] = a;
            }
            dk_g = un.g;
            mma_bar();
        }
    };

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
        if (kFused && k == 0) {
            // both of this CTA's tiles are added up now, at the start, so that every image's flag advances long before
            // any CTA needs dk: the first from the staging buffer, the second from the copy of its interior
            tile_sum(first, stage, SW, P6 * SW + P6, f_red, 0);
            if (!kMany && my_units > 1) {
                if (alive) alive = mbar_wait(boxfull, 0u, p.ctrl, 0xA9000000u);
                tile_sum(first + stride, sumbuf, TW, 0, f_red + kWarps * CG, 1);
            }
            if (kMany) {
                // the later units' interiors, eight rows (one per warp) at a time; a unit's two halves are added in order
                const int gsub = lane >> 3, pr = lane & 7;
                for (int u = 1; u < (int)my_units; ++u) {
                    float keep = 0.f;
#pragma unroll 1
                    for (int half = 0; half < 2; ++half) {
                        const int h = 2 * (u - 1) + half, slot = h & 1;
                        if (alive) alive = mbar_wait(boxfull + 8 * slot, (unsigned)((h >> 1) & 1), p.ctrl, 0xA9000000u);
                        const uint32_t* st32 = reinterpret_cast<const uint32_t*>(sumbuf + slot * (S::BOX_BYTES / 2));
                        float s0 = 0.f, s1 = 0.f;
#pragma unroll
                        for (int i = 0; i < TW / 4; ++i) {
                            const uint32_t v = st32[(warp * TW + 4 * i + gsub) * NPAIR + pr];
                            s0 += __uint_as_float(v << 16);
                            s1 += __uint_as_float(v & 0xffff0000u);
                        }
                        s0 += __shfl_xor_sync(0xffffffffu, s0, 8);  s1 += __shfl_xor_sync(0xffffffffu, s1, 8);
                        s0 += __shfl_xor_sync(0xffffffffu, s0, 16); s1 += __shfl_xor_sync(0xffffffffu, s1, 16);
                        float* fr = f_red + (1 - slot) * (kWarps * CG);      // the first half follows the first tile's sum, which used f_red
                        if (lane < 8) { fr[warp * CG + 2 * lane] = s0; fr[warp * CG + 2 * lane + 1] = s1; }
                        mma_bar();
                        if (tid == 0) mbar_arrive(boxfree0 + 8 * slot);       // everybody is done with the slot
                        if (tid < CG) {
                            float tsum = 0.f;
#pragma unroll
                            for (int w = 0; w < kWarps; ++w) tsum += fr[w * CG + tid];
                            if (half == 0) keep = tsum;
                            else {
                                p.gpart[(first + u * stride) * CG + tid] = keep + tsum;
                                mbar_arrive(sumdone_of(u));
                            }
                        }
                    }
                }
            }
        }
        if (kMix) {                                          // Eq. 5: the depth-wise stage sees F_att * LK^c
            uint32_t mixb[4];
            load_mix_fragments(p.w_point, lane, mixb);
            pointwise_mix_tile<ROWS * SW>(reinterpret_cast<uint32_t*>(stage), mixb, warp, lane);
            fence_async_smem();                              // these stores before the next tile's TMA load into the same buffer
            mma_bar();
        }
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
        if (!kFused && lane == 0) mbar_arrive(empty);        // staging may be refilled
        mma_bar();                                           // planes (and the tap table) complete
        if (kFused && k + 1 < my_units && tid == 0) {        // every warp is past the staging buffer: the next unit's tile
            const Unit nx = decode(first + (k + 1) * stride, p);
            mbar_expect_tx(full, S::STAGE_BYTES);
            tma_load_4d(smem_u32(stage), &map_att, full, nx.g * CG, nx.tx * TW - P6, nx.ty * TH - P6, nx.b);
        }

        // ---- two channels per warp --------------------------------------------------------------------
        // Per channel: 13 kernel rows of tensor-core work into acc / acc1, then the dynamic 3x3 kernel on the CUDA
        // cores, fp32 (Eq. 4 line 3, second term), into dacc; dk is waited for after both channels'
        // tensor-core work.
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
            // Straight-line code for the 13 kernel rows: the loads of a row run ahead of the previous row's products
            // (-4 % on large maps, -1.2 us on a 640x360 forward against the rolled loop).
#pragma unroll
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
            if (kFused) {
#pragma unroll
                for (int v = 0; v < 9; ++v) dkv[v] = f_dk[c * 9 + v];
            } else {
                const float* dp = p.dk + ((size_t)un.b * p.Ca + un.g * CG + c) * 9;
#pragma unroll
                for (int v = 0; v < 9; ++v) dkv[v] = __ldcg(dp + v);
            }
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

        {
            // Both channels' tensor-core work first, then the 3x3 part of each: dk is first needed well after every CTA has
            // arrived for all its tiles (one-launch form) or after the kernel that produces it has run beside this one.
            // (Alternating products and 3x3 part per channel was 4 % slower on large maps.)
            float acc1[NB][NA][4];
            mma_all(acc, warp * 2);
            mma_all(acc1, warp * 2 + 1);
            if (kFused) obtain_dk(un, flag0[kMany ? k : (k == 0 ? 0 : 1)]);
            else if (!dk_ready) { pdl_wait_primary(); dk_ready = true; }
            dk_all(dacc, warp * 2);
            write_back(acc, dacc, warp * 2);
            dk_all(dacc, warp * 2 + 1);
            write_back(acc1, dacc, warp * 2 + 1);
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

// Stage 1 inside the stencil kernel: the estimator's weights and the scratch it needs (see Params).
struct Fused {
    const void *w_last, *b_last, *w_down, *b_down;
    int hidden;
    float* gpart;
    unsigned *garr, *gflag;
};

template <class S, bool kBias, bool kFused, bool kMix = false, bool kMany = false>
inline int launch_shape(int B, int C, int Ca, int H, int W, const void* x, const void* w_large, const float* dk,
                        const float* bias, void* out, unsigned* ctrl, cudaStream_t st, bool dependent, int* launches,
                        std::string* err, const Fused* fu = nullptr, bool skip_copy = false, const void* w_point = nullptr) {
    const int cc = skip_copy ? 0 : C - Ca;                 // skip_copy: the identity channels are consumed elsewhere (fused 1x1)
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
            if (S::TH % shapes[s][1] == 0 && cc * 2 * shapes[s][0] * shapes[s][1] <= (kFused ? 12288 : kMaxSlotBytes)) pick = s;   // one-launch form: its scratch leaves 12 KB per slot
        if (pick < 0) return kNotApplicable;
        p.copy_cw = shapes[pick][0]; p.copy_cr = shapes[pick][1];
        p.slot_stride = (cc * 2 * p.copy_cw * p.copy_cr + 127) / 128 * 128;
    }
    p.w_large = static_cast<const __nv_bfloat16*>(w_large);
    p.w_point = static_cast<const __nv_bfloat16*>(w_point);
    if (kMix && (Ca != CG || !w_point || (reinterpret_cast<uintptr_t>(w_point) & 3u) != 0)) return kNotApplicable;   // one group, 4-byte loads
    p.dk = dk; p.bias = bias; p.out = static_cast<__nv_bfloat16*>(out); p.ctrl = ctrl;
    p.wait_first = dependent ? 0 : 1;
    p.w_last = p.b_last = p.w_down = p.b_down = nullptr; p.hidden = 0; p.gpart = nullptr; p.garr = p.gflag = nullptr;
    p.upi = p.groups * p.tiles_x * p.tiles_y;
    if (kFused) {
        p.w_last = static_cast<const __nv_bfloat16*>(fu->w_last); p.b_last = static_cast<const __nv_bfloat16*>(fu->b_last);
        p.w_down = static_cast<const __nv_bfloat16*>(fu->w_down); p.b_down = static_cast<const __nv_bfloat16*>(fu->b_down);
        p.hidden = fu->hidden; p.gpart = fu->gpart; p.garr = fu->garr; p.gflag = fu->gflag;
    }

    CUtensorMap m_att, m_cin, m_cout, m_box;
    if (!make_map(&m_att, x, B, C, H, W, CG, S::SW, S::ROWS, CU_TENSOR_MAP_L2_PROMOTION_L2_64B)) return kNotApplicable;
    if (!make_map(&m_box, x, B, C, H, W, CG, S::TW, kMany ? S::TH / 2 : S::TH, CU_TENSOR_MAP_L2_PROMOTION_L2_64B)) return kNotApplicable;
    if (cc > 0) {
        if (!make_map(&m_cin, x, B, C, H, W, cc, p.copy_cw, p.copy_cr)) return kNotApplicable;
        if (!make_map(&m_cout, out, B, C, H, W, cc, p.copy_cw, p.copy_cr)) return kNotApplicable;
    } else {
        m_cin = m_att; m_cout = m_att;
    }
    static_assert((S::STAGE_BYTES + CG * S::PLANE_BYTES + PTAB_BYTES) % 128 == 0 && (FUSED_SMEM_FLOATS * 4) % 128 == 0,
                  "the copy ring is a TMA destination: 128-byte aligned");
    const size_t smem = (size_t)S::STAGE_BYTES + (size_t)CG * S::PLANE_BYTES + PTAB_BYTES + (kFused ? FUSED_SMEM_FLOATS * 4 + S::BOX_BYTES : 0) +
                        (size_t)NSLOT * p.slot_stride + 128;  // 128: the mbarriers
    if (smem > 227 * 1024) return kNotApplicable;
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return kNotApplicable;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(stencil_toeplitz_nhwc_bf16<S, kBias, kFused, kMix, kMany>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return kNotApplicable; }
        attr_set[dev] = true;
    }
    const long long grid = p.units < sm_count() ? p.units : sm_count();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeCooperative;             // fused stage 1: CTAs wait on one another, all must be resident
    attr[1].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = kFused ? 2 : 1;
    if (kFused && (grid > sm_count() || p.units > (kMany ? kMaxFusedUnits : 2) * grid)) return kNotApplicable;
    cudaError_t e = cudaLaunchKernelEx(&cfg, stencil_toeplitz_nhwc_bf16<S, kBias, kFused, kMix, kMany>, m_att, m_cin, m_cout, m_box, p);
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
                               cudaStream_t st, bool dependent, int* launches, std::string* err, int* tile_w,
                               bool skip_copy = false, const void* w_point = nullptr) {
    if (!applies(C, Ca, K, dtype, layout) || sm_count() <= 0) return kNotApplicable;
    *tile_w = Shape64x16::TW;
    if (w_point)
        return bias ? kNotApplicable
                    : launch_shape<Shape64x16, false, false, true>(B, C, Ca, H, W, x, w_large, dk, bias, out, ctrl, st, dependent, launches, err, nullptr, skip_copy, w_point);
    return bias ? launch_shape<Shape64x16, true, false>(B, C, Ca, H, W, x, w_large, dk, bias, out, ctrl, st, dependent, launches, err, nullptr, skip_copy)
                : launch_shape<Shape64x16, false, false>(B, C, Ca, H, W, x, w_large, dk, bias, out, ctrl, st, dependent, launches, err, nullptr, skip_copy);
}

// Whether the whole forward can be one launch of the tensor-core kernel with stage 1 inside: the kernel applies,
// no CTA gets more than two units (a CTA adds up its tiles before it needs dk), the estimator fits the scratch.
inline bool fused_applies(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, int hidden) {
    if (!applies(C, Ca, K, dtype, layout) || sm_count() <= 0) return false;
    if (Ca > kFusedMaxCa || hidden > kMaxHidden) return false;
    return units_of<Shape64x16>(B, Ca, H, W) <= (long long)kMaxFusedUnits * sm_count();
}

// The whole forward (stage 1 fused) as one launch; same return convention as try_launch_toeplitz.
inline int try_launch_fused(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x,
                            const void* w_large, const Fused& fu, void* out, unsigned* ctrl, cudaStream_t st,
                            int* launches, std::string* err, int* tile_w, bool skip_copy = false, const void* w_point = nullptr) {
    if (!fused_applies(B, C, Ca, H, W, K, dtype, layout, fu.hidden)) return kNotApplicable;
    *tile_w = Shape64x16::TW;
    const bool many = units_of<Shape64x16>(B, Ca, H, W) > 2LL * sm_count();   // some CTA walks three units or more
    if (w_point)
        return many ? launch_shape<Shape64x16, false, true, true, true>(B, C, Ca, H, W, x, w_large, nullptr, nullptr, out, ctrl, st, /*dependent=*/false,
                                                                        launches, err, &fu, skip_copy, w_point)
                    : launch_shape<Shape64x16, false, true, true>(B, C, Ca, H, W, x, w_large, nullptr, nullptr, out, ctrl, st, /*dependent=*/false,
                                                                  launches, err, &fu, skip_copy, w_point);
    return many ? launch_shape<Shape64x16, false, true, false, true>(B, C, Ca, H, W, x, w_large, nullptr, nullptr, out, ctrl, st, /*dependent=*/false,
                                                                     launches, err, &fu, skip_copy)
                : launch_shape<Shape64x16, false, true>(B, C, Ca, H, W, x, w_large, nullptr, nullptr, out, ctrl, st, /*dependent=*/false,
                                                        launches, err, &fu, skip_copy);
}

}}}  // namespace esc::tma::toep

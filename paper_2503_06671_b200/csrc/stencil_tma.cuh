// Kernel (b), fast path: TMA-staged, register-tiled fused stencil for K = 13 on NHWC bf16 tensors
// (ESC paper, Section 3.3, Eq. 4 lines 3-4, evaluated in the merged form ZP(dk) + LK^s of Eq. 5).
//
// Work unit: a 40x40 output tile of one image for one group of 16 attention channels.  A CTA
// (8 compute warps + 1 copy warp, one CTA per SM, persistent over units) does, per unit:
//   1. one TMA load of the (40+12) x (40+12+1) x 16-channel halo tile; coordinates outside the
//      image are filled with zeros by the TMA unit, which is the 'same' padding;
//   2. 169 taps for a 5x10 output patch per lane, two adjacent channels at a time with packed
//      fp32 FMAs (fma.rn.f32x2): lane = (position q, channel pair p), a warp covers 4 patches x
//      8 pairs.  Kernel rows are visited in the order 0-4, 8-12, 5-7 so that the per-image dynamic
//      taps (rows 5-7 of the merged kernel) are needed last and the wait for the kernel that
//      produces dk costs nothing;
//   3. one rounding to bf16 and 4-byte stores that fill whole 32-byte sectors across 8 lanes.
// Meanwhile the copy warp streams the untouched channels of the same tile global -> shared ->
// global with TMA loads and stores through a small ring, with no register or issue-slot cost.
//
// Shared-memory words of the tile hold one pixel's channel pair (bf16x2); a pixel is 8 words
// (32 bytes), a tile row 53 pixels.  With an odd row pitch and a patch height of 5 the four
// patches of a warp start at pixel indices that differ mod 4, so the 32 lanes of every LDS.32
// hit 32 different banks.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <string>
#include <cstdio>

#include "common.cuh"

namespace esc { namespace tma {

constexpr int kNotApplicable = -1;

constexpr int K13 = 13, P6 = 6;
constexpr int OX = 10, OY = 5;            // outputs per lane: OY rows x OX columns
constexpr int LXP = 4, LYP = 8;           // patches per tile in x and y
constexpr int TW = OX * LXP, TH = OY * LYP;          // 40 x 40 outputs per tile
constexpr int THP = TH + K13 - 1;                    // 52 staged rows
constexpr int PITCH = TW + K13 - 1 + 1;              // 53 staged pixels per row (odd on purpose)
constexpr int CG = 16;                               // channels per unit
constexpr int NPAIR = CG / 2;
constexpr int kComputeWarps = LXP * LYP / 4;         // 8
constexpr int kComputeThreads = kComputeWarps * 32;  // 256
constexpr int kThreads = kComputeThreads + 32;       // + copy warp
constexpr int TILE_BYTES = THP * PITCH * CG * 2;     // 88,192
constexpr int WSM_FLOATS = K13 * 7 * NPAIR * 4;      // [i][jj][pair][4]: taps 2jj,2jj+1 of both channels
constexpr int WSM_BYTES = (WSM_FLOATS * 4 + 127) / 128 * 128;
constexpr int NSLOT = 4, COPY_DEPTH = 3;             // copy ring: slots, loads in flight
constexpr int kMaxSlotBytes = 8192;
constexpr unsigned kSpinLimit = 1u << 22;

static_assert(TILE_BYTES % 128 == 0, "tile buffers must keep 128-byte alignment");
static_assert((OY * PITCH) % 2 == 1, "patch rows must start at distinct pixel indices mod 4");

struct Params {
    int B, C, Ca, H, W;
    int tiles_x, tiles_y, groups;     // units = B * tiles_y * tiles_x * groups
    long long units;
    int copy_cc, copy_cw, copy_cr;    // copy box: channels, pixels, rows (copy_cc == 0: nothing to copy)
    int slot_stride;                  // bytes between ring slots (multiple of 128)
    const __nv_bfloat16* w_large;     // [Ca][13][13]
    const float* dk;                  // [B][Ca][9]
    __nv_bfloat16* out;
    unsigned* ctrl;                   // status words or nullptr
};

// ---- PTX wrappers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls, records where, and lets the caller carry on.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, unsigned parity, unsigned* ctrl, unsigned where) {
    for (unsigned n = 0; n < kSpinLimit; ++n) {
        if (mbar_try_wait(bar, parity)) return true;
        if (n > 64) __nanosleep(64);
    }
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
__device__ __forceinline__ void compute_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kComputeThreads) : "memory"); }

typedef unsigned long long u64;
__device__ __forceinline__ u64 pack2(float lo, float hi) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ void fma2(u64& d, u64 a, u64 b) { asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b)); }

struct Unit { int b, g, ty, tx; };
__device__ __forceinline__ Unit decode_unit(long long u, const Params& p) {
    Unit r;
    r.tx = (int)(u % p.tiles_x); u /= p.tiles_x;
    r.ty = (int)(u % p.tiles_y); u /= p.tiles_y;
    r.g = (int)(u % p.groups);
    r.b = (int)(u / p.groups);
    return r;
}

// Kernel row visited at step s: rows that never see dk first, the three dk rows last.
__device__ __forceinline__ int row_order(int s) { return s < 5 ? s : (s < 10 ? s + 3 : s - 5); }

__global__ void __launch_bounds__(kThreads, 1)
stencil_tma_nhwc_bf16(const __grid_constant__ CUtensorMap map_att, const __grid_constant__ CUtensorMap map_cin,
                      const __grid_constant__ CUtensorMap map_cout, const Params p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    unsigned char* tilebuf = smem;                                   // 2 x TILE_BYTES
    float* wsm = reinterpret_cast<float*>(smem + 2 * TILE_BYTES);    // merged kernel of the current unit
    unsigned char* ring = smem + 2 * TILE_BYTES + WSM_BYTES;         // NSLOT x slot_stride
    u64* bars = reinterpret_cast<u64*>(ring + NSLOT * p.slot_stride);
    const uint32_t full0 = smem_u32(bars), cfull0 = smem_u32(bars + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        mbar_init(full0, 1); mbar_init(full0 + 8, 1);
        for (int s = 0; s < NSLOT; ++s) mbar_init(cfull0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const long long first = blockIdx.x, stride = gridDim.x;

    // ======================= copy warp: untouched channels, TMA in / TMA out ==================
    if (warp == kComputeWarps) {
        if (lane != 0 || p.copy_cc == 0) return;
        const int per_row = TW / p.copy_cw, chunks = per_row * (TH / p.copy_cr);
        const unsigned bytes = (unsigned)(p.copy_cc * p.copy_cw * p.copy_cr * 2);
        long long issued = 0, stored = 0;
        // chunk n of the CTA's stream -> (unit, chunk-in-unit); units with g != 0 copy nothing
        auto coords = [&](long long n, int& cx, int& cy, int& cb) -> bool {
            const long long u = first + (n / chunks) * stride;
            const Unit un = decode_unit(u, p);
            const int ch = (int)(n % chunks);
            cx = un.tx * TW + (ch % per_row) * p.copy_cw;
            cy = un.ty * TH + (ch / per_row) * p.copy_cr;
            cb = un.b;
            return un.g == 0 && cx < p.W && cy < p.H;
        };
        const long long my_units = first < p.units ? (p.units - first + stride - 1) / stride : 0;
        const long long total = my_units * chunks;
        bool alive = true;
        // Software pipeline: the store of chunk n - COPY_DEPTH goes out first, then the load of
        // chunk n is issued, so COPY_DEPTH - 1 loads are always in flight behind it.
        for (long long n = 0; n < total + COPY_DEPTH; ++n) {
            int cx, cy, cb;
            const long long m = n - COPY_DEPTH;
            if (m >= 0 && coords(m, cx, cy, cb)) {
                const int slot = (int)(stored % NSLOT);
                if (alive) alive = mbar_wait(cfull0 + 8 * slot, (unsigned)((stored / NSLOT) & 1), p.ctrl, 0xC0000000u | (unsigned)slot);
                tma_store_4d(&map_cout, smem_u32(ring + slot * p.slot_stride), p.Ca, cx, cy, cb);
                bulk_commit();
                ++stored;
            }
            if (n < total && coords(n, cx, cy, cb)) {
                const int slot = (int)(issued % NSLOT);
                // the store that last used this slot is at least NSLOT - COPY_DEPTH + 1 groups back
                bulk_wait_read<NSLOT - COPY_DEPTH>();
                mbar_expect_tx(cfull0 + 8 * slot, bytes);
                tma_load_4d(smem_u32(ring + slot * p.slot_stride), &map_cin, cfull0 + 8 * slot, p.Ca, cx, cy, cb);
                ++issued;
            }
        }
        bulk_wait_all<0>();
        return;
    }

    // ======================= compute warps ====================================================
    const int q = lane >> 3, pr = lane & 7;                 // patch position in the warp, channel pair
    const int lx = warp & (LXP - 1), ly = (warp >> 2) * 4 + q;
    const int lane_word = ((ly * OY) * PITCH + lx * OX) * NPAIR + pr;

    if (first < p.units && tid == 0) {
        const Unit u0 = decode_unit(first, p);
        mbar_expect_tx(full0, TILE_BYTES);
        tma_load_4d(smem_u32(tilebuf), &map_att, full0, u0.g * CG, u0.tx * TW - P6, u0.ty * TH - P6, u0.b);
    }

    int cur_g = -1;
    bool alive = true;
    long long k = 0;
    for (long long u = first; u < p.units; u += stride, ++k) {
        const Unit un = decode_unit(u, p);
        const int buf = (int)(k & 1);

        // ---- large-kernel taps of this channel group -> shared (fp32, pair-interleaved) -------
        if (un.g != cur_g) {
            if (cur_g >= 0) compute_bar();                  // everyone is done with the old table
            for (int t = tid; t < K13 * 14 * CG; t += kComputeThreads) {
                const int c = t % CG, j = (t / CG) % 14, i = t / (CG * 14);
                float w = 0.f;
                if (j < K13) w = __bfloat162float(p.w_large[((size_t)(un.g * CG + c) * K13 + i) * K13 + j]);
                wsm[((i * 7 + (j >> 1)) * NPAIR + (c >> 1)) * 4 + (j & 1) * 2 + (c & 1)] = w;
            }
            cur_g = un.g;
            compute_bar();
        }

        if (alive) alive = mbar_wait(full0 + 8 * buf, (unsigned)((k >> 1) & 1), p.ctrl, 0xA0000000u | (unsigned)buf);

        u64 acc[OY][OX];
#pragma unroll
        for (int a = 0; a < OY; ++a)
#pragma unroll
            for (int c = 0; c < OX; ++c) acc[a][c] = 0ull;

        const uint32_t* tw = reinterpret_cast<const uint32_t*>(tilebuf + (size_t)buf * TILE_BYTES) + lane_word;

#pragma unroll 1
        for (int s = 0; s < K13; ++s) {
            const int i = row_order(s);
            if (s == 10) {
                // All warps have finished the previous unit (its buffer and its merged rows are free).
                compute_bar();
                if (tid == 0 && u + stride < p.units) {     // prefetch the next unit's tile
                    const Unit nx = decode_unit(u + stride, p);
                    mbar_expect_tx(full0 + 8 * (buf ^ 1), TILE_BYTES);
                    tma_load_4d(smem_u32(tilebuf + (size_t)(buf ^ 1) * TILE_BYTES), &map_att, full0 + 8 * (buf ^ 1),
                                nx.g * CG, nx.tx * TW - P6, nx.ty * TH - P6, nx.b);
                }
                if (k == 0) pdl_wait_primary();             // dk is written by the preceding kernel
                if (tid < CG * 9) {                          // rows 5-7, columns 5-7: LK^s + dk  (Eq. 5)
                    const int c = tid / 9, tap = tid % 9, ii = 5 + tap / 3, jj = 5 + tap % 3;
                    const float w = __bfloat162float(p.w_large[((size_t)(un.g * CG + c) * K13 + ii) * K13 + jj]) +
                                    p.dk[((size_t)un.b * p.Ca + un.g * CG + c) * 9 + tap];
                    wsm[((ii * 7 + (jj >> 1)) * NPAIR + (c >> 1)) * 4 + (jj & 1) * 2 + (c & 1)] = w;
                }
                compute_bar();
            }
            // kernel row i for this lane's channel pair: 13 packed taps
            u64 w[K13];
            {
                const float4* wr = reinterpret_cast<const float4*>(wsm) + (i * 7) * NPAIR + pr;
#pragma unroll
                for (int jj = 0; jj < 7; ++jj) {
                    const float4 v = wr[jj * NPAIR];
                    w[2 * jj] = pack2(v.x, v.y);
                    if (2 * jj + 1 < K13) w[2 * jj + 1] = pack2(v.z, v.w);
                }
            }
            const uint32_t* trow = tw + i * (PITCH * NPAIR);
#pragma unroll
            for (int oy = 0; oy < OY; ++oy) {
                const uint32_t* r = trow + oy * (PITCH * NPAIR);
#pragma unroll
                for (int kk = 0; kk < OX + K13 - 1; ++kk) {
                    const uint32_t v = r[kk * NPAIR];
                    const u64 in = pack2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
#pragma unroll
                    for (int j = 0; j < K13; ++j) {
                        const int ox = kk - j;
                        if (ox >= 0 && ox < OX) fma2(acc[oy][ox], w[j], in);
                    }
                }
            }
        }

        // ---- epilogue: one rounding to bf16, 4-byte stores (8 lanes = one 32-byte sector) -----
        const int y0 = un.ty * TH + ly * OY, x0 = un.tx * TW + lx * OX;
        uint32_t* ow = reinterpret_cast<uint32_t*>(p.out) + un.g * NPAIR + pr;
        const size_t cw = (size_t)p.C / 2;
#pragma unroll
        for (int oy = 0; oy < OY; ++oy) {
            const int y = y0 + oy;
            if (y < p.H) {
                const size_t rowbase = ((size_t)un.b * p.H + y) * p.W;
#pragma unroll
                for (int ox = 0; ox < OX; ++ox) {
                    const int x = x0 + ox;
                    if (x < p.W) {
                        float lo, hi;
                        unpack2(acc[oy][ox], lo, hi);
                        const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
                        ow[(rowbase + x) * cw] = *reinterpret_cast<const uint32_t*>(&h);
                    }
                }
            }
        }
    }
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
inline bool make_map(CUtensorMap* m, const void* base, int B, int C, int H, int W, int bc, int bw, int bh) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    const cuuint32_t box[4] = {(cuuint32_t)bc, (cuuint32_t)bw, (cuuint32_t)bh, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline int sm_count() {
    static int n = []() {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        return v;
    }();
    return n;
}

// Launches the fast kernel if the problem fits it.  Returns 0 on success, kNotApplicable if the
// generic kernel has to run instead, or an ESC_ERR_* code.
inline int try_launch(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x,
                      const void* w_large, const float* dk, void* out, unsigned* ctrl, cudaStream_t st,
                      bool dependent, int* launches, std::string* err) {
    if (K != K13 || dtype != 1 /*bf16*/ || layout != kNHWC) return kNotApplicable;
    if (Ca % CG != 0 || C % 8 != 0) return kNotApplicable;
    const int cc = C - Ca;
    if (cc > 256) return kNotApplicable;
    if (sm_count() <= 0) return kNotApplicable;

    Params p;
    p.B = B; p.C = C; p.Ca = Ca; p.H = H; p.W = W;
    p.tiles_x = (W + TW - 1) / TW; p.tiles_y = (H + TH - 1) / TH; p.groups = Ca / CG;
    p.units = (long long)B * p.groups * p.tiles_x * p.tiles_y;
    p.copy_cc = cc; p.copy_cw = TW; p.copy_cr = 2; p.slot_stride = 128;
    if (cc > 0) {
        static const int shapes[5][2] = {{40, 2}, {40, 1}, {20, 1}, {10, 1}, {5, 1}};
        int pick = -1;
        for (int s = 0; s < 5 && pick < 0; ++s)
            if (cc * 2 * shapes[s][0] * shapes[s][1] <= kMaxSlotBytes) pick = s;
        if (pick < 0) return kNotApplicable;
        p.copy_cw = shapes[pick][0]; p.copy_cr = shapes[pick][1];
        p.slot_stride = (cc * 2 * p.copy_cw * p.copy_cr + 127) / 128 * 128;
    }
    p.w_large = static_cast<const __nv_bfloat16*>(w_large);
    p.dk = dk;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.ctrl = ctrl;

    CUtensorMap m_att, m_cin, m_cout;
    if (!make_map(&m_att, x, B, C, H, W, CG, PITCH, THP)) return kNotApplicable;
    if (cc > 0) {
        if (!make_map(&m_cin, x, B, C, H, W, cc, p.copy_cw, p.copy_cr)) return kNotApplicable;
        if (!make_map(&m_cout, out, B, C, H, W, cc, p.copy_cw, p.copy_cr)) return kNotApplicable;
    } else {
        m_cin = m_att; m_cout = m_att;
    }

    const size_t smem = 128 + 2 * (size_t)TILE_BYTES + WSM_BYTES + (size_t)NSLOT * p.slot_stride + 64;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(stencil_tma_nhwc_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return kNotApplicable; }
        attr_set = true;
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
    cfg.numAttrs = dependent ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, stencil_tma_nhwc_bf16, m_att, m_cin, m_cout, p);
    if (e != cudaSuccess) {
        char buf[256];
        snprintf(buf, sizeof buf, "stencil_tma_nhwc_bf16 launch: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e));
        *err = buf;
        return 7;  // ESC_ERR_CUDA
    }
    ++*launches;
    return 0;
}

}}  // namespace esc::tma

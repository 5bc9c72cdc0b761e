// Kernel (b), tensor-core form, for NCHW bf16 tensors: the K = 13 depth-wise stage of ConvAttn as banded-Toeplitz
// matrix products (ESC paper, Section 3.3, Eq. 4 lines 3-4), the arithmetic of stencil_toeplitz.cuh on the layout
// in which the instruction's operands need no transposition:
//
//   D (16 x-outputs  x  8 rows)  +=  A (16 x 16: Toeplitz block, weights)  x  B (16 x-inputs x 8 rows: image)
//
// NCHW keeps a channel's rows x-contiguous, so a unit's halo tile -- 16 channels x 28 rows x 88 columns -- lands by
// ONE TMA load directly as the 16 planes the tensor-core loop reads (row pitch 88 elements = 8 x odd: the eight rows
// of an ldmatrix fall in different bank groups; zero fill = the padding), in one of two buffers, so that the next
// unit's tile is in flight while this one is worked on.  A TMA load starts on a 16-byte boundary: the tile starts
// 8 columns (not 6) left of its first output, and the Toeplitz band is shifted by two taps instead.  Results go
// back into the plane and leave as 128-byte row segments, one coalesced 4-byte store per lane, straight from the
// warp that computed the channel: no block-wide barrier per unit.  The identity channels of an image are one
// contiguous range: the copy warp moves it in 16 KB pieces with plain bulk copies (global -> shared -> global).
//
// One CTA per SM, persistent over units (64 x 16 outputs x 16 channels of one image):
//   warps 0-7   two channels each: 13 kernel rows x 5 input blocks on the tensor cores, the dynamic 3x3 kernel in
//               fp32 on the CUDA cores (dk is an fp32 quantity), one rounding to bf16, stores
//   warp 8      tile producer (TMA); with stage 1 inside the kernel also the arrivals on the images' counters
//   warp 9      copy-through of the untouched channels
// kFused: stage 1 of the module (Eq. 4 line 2) inside this kernel, as in the NHWC kernel: every CTA adds up the
// interiors of its (at most two) tiles, arrives on the image's counter, the last arrival advances the image's
// flag, and every CTA then evaluates the estimator for the channels it works on.  Cooperative launch, bounded waits.
#pragma once
#include "stencil_toeplitz.cuh"

namespace esc { namespace tma { namespace toepn {

using toep::kWarps; using toep::kMmaThreads; using toep::kThreads; using toep::PT; using toep::PTAB_BYTES;
using toep::ldsm_x4; using toep::mma_bf16; using toep::mma_bar; using toep::ld_acquire; using toep::st_release;
using toep::kFusedMaxCa; using toep::kFlagPolls; using toep::FUSED_SMEM_FLOATS;

constexpr int TH = 16, TW = 64, NA = 2, NB = 4;
constexpr int ROWS = TH + K13 - 1;                  // 28 staged rows
constexpr int XS = 8;                               // staged columns left of the first output (a multiple of 8: 16 bytes)
constexpr int PP = 88;                              // staged columns = plane row pitch: XS + TW + 6, rounded up to 8 x odd
constexpr int PLANE = ROWS * PP * 2;                // 4,928 bytes
constexpr int BUF_BYTES = CG * PLANE;               // 78,848: a TMA destination, a multiple of 128
constexpr int kCopySlots = 3, kCopySlotBytes = 16384;
static_assert(PP % 8 == 0 && (PP / 8) % 2 == 1 && PP >= XS + TW + P6 && BUF_BYTES % 128 == 0, "plane geometry");
static_assert(16 * (NB + 1) + 8 <= PP, "the last input block's ldmatrix stays inside a plane row");

struct Params {
    int B, C, Ca, H, W;
    int tiles_x, tiles_y, groups;
    long long units;
    const __nv_bfloat16* x;           // for the copy-through
    const __nv_bfloat16* w_large;     // [Ca][13][13]
    const __nv_bfloat16* w_point;     // kMix: [16][16] point-wise filter LK^c of the decomposed form (Eq. 5), row = output channel
    const float* dk;                  // [B][Ca][9]
    const float* bias;                // [B][Ca] constant added to every output of (image, channel), or nullptr (backward pass)
    __nv_bfloat16* out;
    unsigned* ctrl;
    int wait_first;
    long long copy_bytes;             // identity channels of one image, bytes (0: nothing to copy)
    // stage 1 inside the kernel (see stencil_toeplitz.cuh)
    const __nv_bfloat16 *w_last, *b_last, *w_down, *b_down;
    int hidden;
    float* gpart;
    unsigned *garr, *gflag;
    int upi;
};

__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, unsigned bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src, unsigned bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}

__device__ __forceinline__ Unit decode(long long u64v, const Params& p) {
    unsigned u = (unsigned)u64v;
    Unit r;
    r.tx = (int)(u % (unsigned)p.tiles_x); u /= (unsigned)p.tiles_x;
    r.ty = (int)(u % (unsigned)p.tiles_y); u /= (unsigned)p.tiles_y;
    r.g = (int)(u % (unsigned)p.groups);
    r.b = (int)(u / (unsigned)p.groups);
    return r;
}

__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}

// kMix: the decomposed large kernel of Eq. 5 -- after a tile has landed (and, with stage 1 inside, after its sum has been
// taken from the unmixed values) the 16 planes are replaced, eight pixels at a time and in place, by LK^c applied across
// them: D (16 output channels x 8 pixels) = LK^c (16 x 16) x B (16 channels x 8 pixels), B straight from the planes by
// ldmatrix.trans, one rounding to bf16; then one block-wide barrier before the depth-wise products.
template <bool kFused, bool kMix = false>
__global__ void __launch_bounds__(kThreads, 1)
stencil_toeplitz_nchw_bf16(const __grid_constant__ CUtensorMap map_att, const Params p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* bufs = smem;                                                    // 2 x 16 planes [ROWS][PP] bf16
    uint32_t* ptab = reinterpret_cast<uint32_t*>(smem + 2 * BUF_BYTES);            // [16][13][PT] packed tap pairs
    float* fsm = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(ptab) + PTAB_BYTES);   // stage 1 scratch
    unsigned char* ring = reinterpret_cast<unsigned char*>(fsm) + FUSED_SMEM_FLOATS * 4;
    u64* bars = reinterpret_cast<u64*>(ring + kCopySlots * kCopySlotBytes);
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 16, cfull0 = empty0 + 16, sumdone = cfull0 + 8 * kCopySlots;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, kWarps); }
        for (int s = 0; s < kCopySlots; ++s) mbar_init(cfull0 + 8 * s, 1);
        mbar_init(sumdone, kWarps);                          // one barrier per unit (the producer lane may fall behind by more
        mbar_init(sumdone + 8, kWarps);                      // than the one phase a parity wait can tell apart)
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
            // ---- tile producer: buffer k & 1 is free again once every warp has stored the results of unit k - 2
            bool alive = true;
            unsigned seen[2] = {0u, 0u};
            for (long long k = 0; k < my_units; ++k) {
                const int buf = (int)(k & 1);
                if (k >= 2 && alive) alive = mbar_wait(empty0 + 8 * buf, (unsigned)(((k >> 1) - 1) & 1), p.ctrl, 0xB8000000u);
                const Unit un = decode(first + k * stride, p);
                mbar_expect_tx(full0 + 8 * buf, BUF_BYTES);
                tma_load_4d(smem_u32(bufs + buf * BUF_BYTES), &map_att, full0 + 8 * buf, un.tx * TW - XS, un.ty * TH - P6, un.g * CG, un.b);
                // the flags as they stand before this CTA arrives anywhere: they cannot have advanced yet
                if (kFused && k < 2) seen[k] = ld_acquire(p.gflag + un.b);
            }
            if (kFused) {
                // arrivals on the images' counters once the working warps have written a unit's 16 sums; the atomic's
                // round trip stays off their path
                for (int k = 0; k < (int)my_units && k < 2; ++k) {
                    const Unit un = decode(first + k * stride, p);
                    if (alive) alive = mbar_wait(sumdone + 8 * k, 0u, p.ctrl, 0xB9000000u);
                    unsigned old;
                    asm volatile("atom.acq_rel.gpu.global.inc.u32 %0, [%1], %2;" : "=r"(old) : "l"(p.garr + un.b), "r"((unsigned)(p.upi - 1)) : "memory");
                    if (old == (unsigned)(p.upi - 1)) st_release(p.gflag + un.b, seen[k] + 1u);   // the counter has wrapped back to 0
                }
            }
        } else if (p.copy_bytes != 0) {
            // ---- copy-through: the identity channels of image b are the contiguous range that starts at channel Ca
            const long long per_img = (p.copy_bytes + kCopySlotBytes - 1) / kCopySlotBytes, total = per_img * p.B;
            const long long mine = first < total ? (total - first + stride - 1) / stride : 0;
            const size_t img_elems = (size_t)p.C * p.H * p.W, skip = (size_t)p.Ca * p.H * p.W;
            auto place = [&](long long n, size_t* off, unsigned* bytes) {
                const long long ch = first + n * stride, b = ch / per_img, piece = ch - b * per_img;
                const long long at = piece * kCopySlotBytes, left = p.copy_bytes - at;
                *off = (size_t)b * img_elems + skip + (size_t)(at / 2);
                *bytes = (unsigned)(left < kCopySlotBytes ? left : kCopySlotBytes);
            };
            auto issue = [&](long long n) {
                size_t off; unsigned bytes;
                place(n, &off, &bytes);
                const int slot = (int)(n % kCopySlots);
                bulk_wait_read<1>();                          // the store that last read this slot (piece n - 3) is done with it
                mbar_expect_tx(cfull0 + 8 * slot, bytes);
                bulk_g2s(smem_u32(ring + slot * kCopySlotBytes), p.x + off, bytes, cfull0 + 8 * slot);
            };
            bool alive = true;
            if (mine > 0) issue(0);
            for (long long n = 0; n < mine; ++n) {
                if (n + 1 < mine) issue(n + 1);
                size_t off; unsigned bytes;
                place(n, &off, &bytes);
                const int slot = (int)(n % kCopySlots);
                if (alive) alive = mbar_wait(cfull0 + 8 * slot, (unsigned)((n / kCopySlots) & 1), p.ctrl, 0xC8000000u | (unsigned)slot);
                bulk_s2g(p.out + off, smem_u32(ring + slot * kCopySlotBytes), bytes);
                bulk_commit();
            }
            bulk_wait_all<0>();
        }
        return;
    }

    // ======================= the eight working warps ===============================================
    const int g = lane >> 2, t = lane & 3;
    const int mi = lane >> 3, mr = lane & 7;
    // This lane's packed tap pairs P[e], P[e + 8], P[e + 16]; the tile starts XS - 6 = 2 columns early, hence e = 2t - g - 2.
    const int e0 = 2 * t - g - (XS - P6);
    const int ia = min(max(e0, -2), 13) + 2, ib = min(max(e0 + 8, -2), 13) + 2, ic = min(max(e0 + 16, -2), 13) + 2;

    int cur_g = -1;
    bool alive = true, dk_ready = p.wait_first != 0;

    // ---- stage 1 inside the kernel --------------------------------------------------------------------
    float* f_sub = fsm;                                      // [256] sub-sums of the partial sums
    float* f_mean = fsm + kMmaThreads;                       // [Ca] pooled means of the current image
    float* f_act = f_mean + kFusedMaxCa;                     // [hidden] activations of the two-layer estimator
    float* f_dk = f_act + kMaxHidden;                        // [16][9] dynamic taps of the current (image, group)
    unsigned flag0[2] = {0u, 0u};
    int dk_b = -1, dk_g = -1;
    if (kFused) {
        for (int k = 0; k < (int)my_units && k < 2; ++k) flag0[k] = ld_acquire(p.gflag + decode(first + k * stride, p).b);
    }
    // Sum of a tile's interior (the tiles' interiors partition the image; pixels outside it are zero-filled): this
    // warp's two channels, a row of 64 pixels per load, rows in order, then a fixed butterfly over the lanes.
    auto tile_sum = [&](const long long unit_index, const unsigned char* buf, const int k_of_cta) {
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
            const uint32_t* pl = reinterpret_cast<const uint32_t*>(buf + (size_t)(warp * 2 + cc) * PLANE) + (P6 * PP + XS) / 2 + lane;
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
            if (lane == 0) p.gpart[unit_index * CG + warp * 2 + cc] = s;
        }
        if (lane == 0) mbar_arrive(sumdone + 8 * k_of_cta);
    };
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
                for (int tl = sub; tl < tpi; tl += 16 * nsub) {
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
        } else {
            mma_bar();                                       // the previous group's taps have been read by everybody
        }
        {
            const float* vin = p.hidden > 0 ? f_act : f_mean;
            const int n_in = p.hidden > 0 ? p.hidden : p.Ca;
            if (tid < CG * 9) {
                const int o = un.g * CG * 9 + tid;
                float a = __bfloat162float(p.b_last[o]);
                const __nv_bfloat16* wr = p.w_last + (size_t)o * n_in;
                for (int c0 = 0; c0 < n_in; c0 += 16) {
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
        const int bufi = (int)(k & 1);
        unsigned char* planes = bufs + bufi * BUF_BYTES;
        const uint32_t planes_a = smem_u32(planes);

        // ---- packed tap pairs of this channel group: P[c][i][d + 2] = (LK[c][i][d], LK[c][i][d + 1]), zero outside 0..12
        if (un.g != cur_g) {
            if (cur_g >= 0) mma_bar();                       // everybody is done with the old table
            const unsigned short* wg = reinterpret_cast<const unsigned short*>(p.w_large) + (size_t)un.g * CG * K13 * K13;
            constexpr int N = CG * K13 * PT, PER = N / kMmaThreads;
            static_assert(N % kMmaThreads == 0, "table entries per thread");
            unsigned lo[PER], hi[PER];
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int e = tid + u * kMmaThreads, d = (e % PT) - 2, row = e / PT;   // row = c * 13 + i
                lo[u] = (d >= 0 && d < K13) ? wg[row * K13 + d] : 0u;
                hi[u] = (d + 1 >= 0 && d + 1 < K13) ? wg[row * K13 + d + 1] : 0u;
            }
#pragma unroll
            for (int u = 0; u < PER; ++u) ptab[tid + u * kMmaThreads] = lo[u] | (hi[u] << 16);
            cur_g = un.g;
            mma_bar();
        }

        // ---- the tile has landed: it is the 16 planes -------------------------------------------------------
        if (alive) alive = mbar_wait(full0 + 8 * bufi, (unsigned)((k >> 1) & 1), p.ctrl, 0xA8000000u);
        if (kFused && k == 0) {
            // both of this CTA's tiles are added up now, at the start, so that every image's flag advances long before
            // any CTA needs dk
            tile_sum(first, planes, 0);
            if (my_units > 1) {
                if (alive) alive = mbar_wait(full0 + 8, 0u, p.ctrl, 0xA9000000u);
                tile_sum(first + stride, bufs + BUF_BYTES, 1);
            }
        }

        if (kMix) {
            // A = LK^c: a0 = (row g, columns 2t, 2t + 1), a1 = (row g + 8, ...), a2 / a3 = the same rows, columns + 8
            const uint32_t* wp = reinterpret_cast<const uint32_t*>(p.w_point);
            const uint32_t a0 = __ldg(wp + g * 8 + t), a1 = __ldg(wp + (g + 8) * 8 + t);
            const uint32_t a2 = __ldg(wp + g * 8 + 4 + t), a3 = __ldg(wp + (g + 8) * 8 + 4 + t);
            constexpr int BPR = PP / 8, NBLK = ROWS * BPR;   // blocks of 8 pixels per row, per plane
            for (int pb = 2 * warp; pb < NBLK; pb += 2 * kWarps) {
                // matrix mi: channels 8 (mi & 1) .. + 7 of pixel block pb + (mi >> 1); row mr of it = one channel's 8 pixels
                const int blk = min(pb + (mi >> 1), NBLK - 1);
                const uint32_t at = (uint32_t)(((mi & 1) * 8 + mr) * PLANE + ((blk / BPR) * PP + (blk % BPR) * 8) * 2);
                uint32_t b[4];
                ldsm_x4_trans(planes_a + at, b);
                float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
                mma_bf16(d0, a0, a1, a2, a3, b[0], b[1]);
                mma_bf16(d1, a0, a1, a2, a3, b[2], b[3]);
                __syncwarp();                                // every lane has its inputs before any plane is overwritten
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int bk = pb + h;
                    if (bk < NBLK) {
                        const float* d = h ? d1 : d0;
                        unsigned char* px = planes + ((size_t)(bk / BPR) * PP + (bk % BPR) * 8 + 2 * t) * 2;
                        const __nv_bfloat162 lo = __floats2bfloat162_rn(d[0], d[1]), hi = __floats2bfloat162_rn(d[2], d[3]);
                        *reinterpret_cast<__nv_bfloat162*>(px + (size_t)g * PLANE) = lo;
                        *reinterpret_cast<__nv_bfloat162*>(px + (size_t)(g + 8) * PLANE) = hi;
                    }
                }
            }
            fence_async_smem();                              // these stores before the next tile's TMA load into the same buffer
            mma_bar();                                       // every plane is mixed before any warp multiplies
        }
        const unsigned sh = (g & 1) ? 0u : 16u;
        float acc[NB][NA][4], acc1[NB][NA][4], dacc[NB][NA][4];
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
#pragma unroll
            for (int i = 0; i < K13; ++i) {
                const uint32_t pa = pt[i * PT + ia], pb = pt[i * PT + ib], pc = pt[i * PT + ic];
                // A0[m][k] = LK[i][k - m - 2] (outputs of block q from inputs of block q),
                // A1[m][k] = LK[i][k - m + 14] (outputs of block q - 1 from inputs of block q)
#pragma unroll
                for (int q = 0; q <= NB; ++q) {
                    uint32_t b[4];
                    ldsm_x4(b_lane + (uint32_t)((i * PP + 16 * q) * 2), b);
                    if (q < NB) {
                        mma_bf16(a4[q][0], pa, 0u, pb, pa, b[0], b[1]);
                        mma_bf16(a4[q][1], pa, 0u, pb, pa, b[2], b[3]);
                    }
                    if (q >= 1) {
                        mma_bf16(a4[q - 1][0], pc, pb, 0u, pc, b[0], b[1]);
                        mma_bf16(a4[q - 1][1], pc, pb, 0u, pc, b[2], b[3]);
                    }
                }
            }
        };
        // 3x3 for outputs (x = 16q + 8h + g, y = 8r + 2t) and (x, y + 1): the three inputs x - 1 .. x + 1 are the
        // staged columns x + 7 .. x + 9, in two aligned 32-bit words; which halves depends on the parity of g alone.
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
            const float bias = p.bias ? __ldg(p.bias + (size_t)un.b * p.Ca + un.g * CG + c) : 0.f;
#pragma unroll
            for (int q = 0; q < NB; ++q)
#pragma unroll
                for (int r = 0; r < NA; ++r)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int wi = (16 * q + 8 * h + g + XS - 1) >> 1, y = 8 * r + 2 * t;
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
        // result of channel c = acc + dacc, rounded once to bf16, into rows 0 .. TH-1, columns 0 .. TW-1 of its plane,
        // and from there to the output as rows of 64 pixels: 128 contiguous bytes per store instruction
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
            __syncwarp();
            const int px = un.tx * TW + 2 * lane, y0 = un.ty * TH;
            if (px < p.W) {                                  // W is even: a pair of pixels is inside or outside together
                __nv_bfloat16* dst = p.out + (((size_t)un.b * p.C + un.g * CG + c) * p.H + y0) * p.W + px;
                const uint32_t* src = reinterpret_cast<const uint32_t*>(plane) + lane;
#pragma unroll
                for (int r = 0; r < TH; ++r)
                    if (y0 + r < p.H) *reinterpret_cast<uint32_t*>(dst + (size_t)r * p.W) = src[r * (PP / 2)];
            }
        };

        // Both channels' tensor-core work first, then the 3x3 part of each: dk is first needed well after every CTA has
        // arrived for all its tiles (one-launch form) or after the kernel that produces it has run beside this one.
        mma_all(acc, warp * 2);
        mma_all(acc1, warp * 2 + 1);
        if (kFused) obtain_dk(un, flag0[k == 0 ? 0 : 1]);
        else if (!dk_ready) { pdl_wait_primary(); dk_ready = true; }
        dk_all(dacc, warp * 2);
        write_back(acc, dacc, warp * 2);
        dk_all(dacc, warp * 2 + 1);
        write_back(acc1, dacc, warp * 2 + 1);
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * bufi);       // this warp is done with the buffer
    }
}

// ---- host side ------------------------------------------------------------------------------
inline bool make_map_nchw(CUtensorMap* m, const void* base, int B, int C, int H, int W) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)C, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)W * 2, (cuuint64_t)H * W * 2, (cuuint64_t)C * H * W * 2};
    const cuuint32_t box[4] = {(cuuint32_t)PP, (cuuint32_t)ROWS, (cuuint32_t)CG, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline long long units_of(int B, int Ca, int H, int W) {
    return (long long)B * (Ca / CG) * ((W + TW - 1) / TW) * ((H + TH - 1) / TH);
}

// bf16 NCHW, K = 13, whole groups of 16 attention channels, rows a multiple of 16 bytes (a TMA stride), 16-byte
// aligned tensors (a TMA base, and the bulk copies of the identity channels).
inline bool applies(int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x, const void* out) {
    (void)H;
    return K == K13 && dtype == 1 /*bf16*/ && layout == kNCHW && Ca % CG == 0 && C >= Ca && W % 8 == 0 &&
           (reinterpret_cast<uintptr_t>(x) & 15u) == 0 && (reinterpret_cast<uintptr_t>(out) & 15u) == 0;
}

template <bool kFused, bool kMix = false>
inline int launch(int B, int C, int Ca, int H, int W, const void* x, const void* w_large, const float* dk, const float* bias, void* out,
                  unsigned* ctrl, cudaStream_t st, bool dependent, int* launches, std::string* err, const toep::Fused* fu,
                  const void* w_point = nullptr, bool skip_copy = false) {
    Params p;
    p.B = B; p.C = C; p.Ca = Ca; p.H = H; p.W = W;
    p.tiles_x = (W + TW - 1) / TW; p.tiles_y = (H + TH - 1) / TH; p.groups = Ca / CG;
    p.units = units_of(B, Ca, H, W);
    if (p.units > 0x7fffffffLL) return kNotApplicable;
    p.x = static_cast<const __nv_bfloat16*>(x);
    p.w_large = static_cast<const __nv_bfloat16*>(w_large);
    p.w_point = static_cast<const __nv_bfloat16*>(w_point);
    if (kMix && (Ca != CG || !w_point || (reinterpret_cast<uintptr_t>(w_point) & 3u) != 0)) return kNotApplicable;   // one group, 4-byte loads
    p.dk = dk; p.bias = bias; p.out = static_cast<__nv_bfloat16*>(out); p.ctrl = ctrl;
    p.wait_first = dependent ? 0 : 1;
    p.copy_bytes = skip_copy ? 0 : (long long)(C - Ca) * H * W * 2;   // a multiple of 16: W is a multiple of 8; skip_copy: consumed elsewhere (fused 1x1)
    p.w_last = p.b_last = p.w_down = p.b_down = nullptr; p.hidden = 0; p.gpart = nullptr; p.garr = p.gflag = nullptr;
    p.upi = p.groups * p.tiles_x * p.tiles_y;
    if (kFused) {
        p.w_last = static_cast<const __nv_bfloat16*>(fu->w_last); p.b_last = static_cast<const __nv_bfloat16*>(fu->b_last);
        p.w_down = static_cast<const __nv_bfloat16*>(fu->w_down); p.b_down = static_cast<const __nv_bfloat16*>(fu->b_down);
        p.hidden = fu->hidden; p.gpart = fu->gpart; p.garr = fu->garr; p.gflag = fu->gflag;
    }
    CUtensorMap m_att;
    if (!make_map_nchw(&m_att, x, B, C, H, W)) return kNotApplicable;
    static_assert((2 * BUF_BYTES + PTAB_BYTES + FUSED_SMEM_FLOATS * 4) % 128 == 0, "the copy ring is a bulk-copy destination");
    const size_t smem = (size_t)2 * BUF_BYTES + PTAB_BYTES + FUSED_SMEM_FLOATS * 4 + (size_t)kCopySlots * kCopySlotBytes + 128;  // 128: the mbarriers
    static_assert((size_t)2 * BUF_BYTES + PTAB_BYTES + FUSED_SMEM_FLOATS * 4 + (size_t)kCopySlots * kCopySlotBytes + 128 <= 227 * 1024, "shared memory");
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return kNotApplicable;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(stencil_toeplitz_nchw_bf16<kFused, kMix>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
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
    attr[1].id = cudaLaunchAttributeCooperative;             // stage 1 inside: CTAs wait on one another, all must be resident
    attr[1].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = kFused ? 2 : 1;
    if (kFused && (grid > sm_count() || p.units > 2 * grid)) return kNotApplicable;
    cudaError_t e = cudaLaunchKernelEx(&cfg, stencil_toeplitz_nchw_bf16<kFused, kMix>, m_att, p);
    if (e != cudaSuccess) {
        char buf[256];
        snprintf(buf, sizeof buf, "stencil_toeplitz_nchw_bf16 launch: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e));
        *err = buf;
        return 7;  // ESC_ERR_CUDA
    }
    ++*launches;
    return 0;
}

// Launches the NCHW tensor-core stencil if the problem fits it: 0 on success, kNotApplicable otherwise, or an ESC_ERR_* code.
inline int try_launch(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x, const void* w_large,
                      const float* dk, const float* bias, void* out, unsigned* ctrl, cudaStream_t st, bool dependent,
                      int* launches, std::string* err, const void* w_point = nullptr, bool skip_copy = false) {
    if (!applies(C, Ca, H, W, K, dtype, layout, x, out) || sm_count() <= 0) return kNotApplicable;
    if (w_point)
        return bias ? kNotApplicable
                    : launch<false, true>(B, C, Ca, H, W, x, w_large, dk, bias, out, ctrl, st, dependent, launches, err, nullptr, w_point, skip_copy);
    return launch<false>(B, C, Ca, H, W, x, w_large, dk, bias, out, ctrl, st, dependent, launches, err, nullptr, nullptr, skip_copy);
}

inline bool fused_applies(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, int hidden, const void* x, const void* out) {
    if (!applies(C, Ca, H, W, K, dtype, layout, x, out) || sm_count() <= 0) return false;
    if (Ca > kFusedMaxCa || hidden > kMaxHidden) return false;
    return units_of(B, Ca, H, W) <= 2LL * sm_count();
}

// The whole forward (stage 1 inside) as one launch.
inline int try_launch_fused(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x, const void* w_large,
                            const toep::Fused& fu, void* out, unsigned* ctrl, cudaStream_t st, int* launches, std::string* err,
                            const void* w_point = nullptr, bool skip_copy = false) {
    if (!fused_applies(B, C, Ca, H, W, K, dtype, layout, fu.hidden, x, out)) return kNotApplicable;
    if (w_point)
        return launch<true, true>(B, C, Ca, H, W, x, w_large, nullptr, nullptr, out, ctrl, st, /*dependent=*/false, launches, err, &fu, w_point, skip_copy);
    return launch<true>(B, C, Ca, H, W, x, w_large, nullptr, nullptr, out, ctrl, st, /*dependent=*/false, launches, err, &fu, nullptr, skip_copy);
}

}}}  // namespace esc::tma::toepn

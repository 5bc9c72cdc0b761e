// Dense large kernel (ESC paper, Section 3.2: LK in R^{13x13x16x16}; Eq. 4 line 3 with that LK) for NHWC bf16
// tensors with 16 attention channels on the fifth-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory):
//
//   out[b,n,y,x] = sum_{k,i,j} w_dense[n,k,i,j] x[b,k,y+i-6,x+j-6]  +  sum_{i,j} dk[b,n,i,j] x[b,n,y+i-1,x+j-1]
//
// Formulation.  One INPUT row of a 128-pixel-wide strip, shifted by a tap column j, is the A operand
// (M = 128 pixels, K = 16 input channels) of ONE instruction whose B operand stacks all 13 kernel rows:
// B_j[k][(12 - i) * 16 + n] = w_dense[n][k][i][j], N = 13 x 16 = 208.  Column block c of the result belongs to
// output row (input row) - 6 + c, so the accumulators of 32 output rows live side by side in the 512 columns
// of tensor memory (row y in columns (y mod 32) * 16 ..) and an input row is used once -- 13 instructions,
// one per tap column -- and never again.  Per instruction 128 x 208 x 16 multiply-adds against 4 KB + 6.5 KB
// of shared-memory operands: the tensor pipe, not shared memory, is the bound, and nothing is unfolded.
// At the ends of a CTA's row range the instruction takes only the column blocks that exist (N = 16 .. 192).
//
// Operands are K-major.  A: a staged input row is [pixel][16 channels], 32 bytes per pixel, written by ONE TMA load
// per row (zero fill = the padding) with the 32-byte swizzle, and described to the tensor core with the same
// swizzle; the swizzle is a function of the shared-memory address, so the descriptor may start at ANY pixel and
// the tap column j is a shift of its start address by 32 * j bytes (verified output by output against
// a direct fp64 evaluation).  B: the weights, without swizzle ([half of K][row][8 k-values], rows 16 bytes apart).
// What bounds it: an instruction takes about 110-130 cycles whatever its N, so the 12 input rows above and below
// a CTA's range, which feed only some of the 13 column blocks, cost as much as full rows: with 13 output rows per
// CTA (640x360 on 148 SMs) 25 row-times are spent for 13 rows of results; larger maps give longer ranges.
//
// Roles (224 threads, one CTA per SM, each CTA one range of rows of one strip):
//   warp 0   lane 0 requests input rows by TMA (one load per row) into a ring of 16; the warp allocates and frees tensor memory
//   warp 1   lane 0 issues the instructions and commits them to mbarriers (ring slot consumed / output row complete)
//   warps 2-5  epilogue: tcgen05.ld of a finished row (one pixel per thread, 16 channels), the dynamic 3x3
//            kernel in fp32 on the CUDA cores from the same ring, one rounding to bf16, 32-byte store;
//            the row's columns are cleared for their next user.
//   warp 6   lane 0 copies the identity channels of the CTA's rows, TMA in / TMA out through a ring of two slots.
#pragma once
#include "stencil_generic.cuh"
#include "stencil_tma.cuh"

namespace esc { namespace tma { namespace umma {

constexpr int MW = 128;                       // output pixels per strip row = M of the instruction
constexpr int SPX = 144;                      // staged pixels per row: 128 + 12, padded to keep half-rows 128-byte aligned
constexpr int HALF_BYTES = SPX * 16;
constexpr int ROW_BYTES = 2 * HALF_BYTES;     // one staged row: SPX pixels x 32 bytes
constexpr int NRING = 16;                     // input rows in flight / kept for the 3x3 part
constexpr int NBLK = K13;                     // column blocks of 16 (kernel rows) in a B operand
constexpr int BHALF_BYTES = NBLK * CG * 16;   // 3,328: one tap column, one channel half: [208 rows][8 k]
constexpr int BJ_BYTES = 2 * BHALF_BYTES;
constexpr int B_BYTES = K13 * BJ_BYTES;       // 86,528
constexpr int SLOTS = 32;                     // output rows whose accumulators fit tensor memory (512 columns)
constexpr int kThreads = 224;                 // producer, issuer, four epilogue warps, copy-through warp
constexpr int kEpiThreads = 128;
constexpr int kCopySlotBytes = 16384, kCopySlots = 2;
constexpr unsigned kPollLimit = 1u << 22;
constexpr int kMiscBytes = 1024;               // dk, progress word, tensor-memory base
constexpr int kBarBytes = 1024;                // 2 * NRING + SLOTS + kCopySlots mbarriers
constexpr int kCopyRingOffset = NRING * ROW_BYTES + B_BYTES + kMiscBytes + kBarBytes;
constexpr size_t kSmemBytes = (size_t)kCopyRingOffset + kCopySlots * kCopySlotBytes;
static_assert((2 * NRING + SLOTS + kCopySlots) * 8 <= kBarBytes && kCopyRingOffset % 128 == 0, "barriers fit; the copy ring is a TMA destination");
static_assert(HALF_BYTES % 128 == 0, "TMA destinations are 128-byte aligned");

struct Params {
    int B, C, H, W;
    int strips, segs, seg_rows;       // per image: strips of 128 pixels x row ranges of seg_rows rows
    const __nv_bfloat16* w_dense;     // [16][16][13][13]  (output channel, input channel, row, column)
    const float* dk;                  // [B][16][9]
    __nv_bfloat16* out;
    unsigned* ctrl;
    int wait_first;
    int w_aligned;                    // w_dense is 16-byte aligned: the B operands are built from a staged copy
    int copy_cc, copy_pw;             // identity channels; pixels of a strip row per copy chunk (0: nothing to copy)
};

// Shared-memory matrix descriptor, K-major, no swizzle: 8 rows x 16 bytes are contiguous (rows 16 bytes apart),
// the next 8 rows follow `sbo` bytes on, the second half of K (k = 8..15) `lbo` bytes on.
__device__ __forceinline__ unsigned long long smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (unsigned long long)((addr >> 4) & 0x3FFFu) | ((unsigned long long)((lbo >> 4) & 0x3FFFu) << 16) |
           ((unsigned long long)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// A operand: K-major with the 32-byte swizzle -- a row (pixel) is 32 contiguous bytes, its two 16-byte halves swapped
// where bit 7 of the shared-memory address is set -- exactly what a TMA load with CU_TENSOR_MAP_SWIZZLE_32B writes for
// a 32-byte inner box.  Rows are 32 bytes apart, 8-row groups 256 bytes.
__device__ __forceinline__ unsigned long long smem_desc_sw32(uint32_t addr) {
    return (unsigned long long)((addr >> 4) & 0x3FFFu) | (1ull << 16) | ((unsigned long long)(256u >> 4) << 32) | (1ull << 46) |
           (6ull << 61);
}
// Instruction descriptor of kind::f16: D fp32, A and B bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(MW >> 4) << 24);
}
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, unsigned long long da, unsigned long long db, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_zero16(uint32_t taddr) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
                 ::"r"(taddr), "r"(0u) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire_cta(const int* p) {
    int v;
    asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_cta(int* p, int v) {
    asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
    tma_load_4d(dst, map, bar, c0, c1, c2, c3);
}

__global__ void __launch_bounds__(kThreads, 1)
stencil_dense_umma_nhwc_bf16(const __grid_constant__ CUtensorMap map_half, const __grid_constant__ CUtensorMap map_cin,
                             const __grid_constant__ CUtensorMap map_cout, const Params p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* ring = smem;                                             // [NRING][SPX pixels][32 bytes], 32-byte swizzle
    unsigned char* btab = smem + NRING * ROW_BYTES;                         // [13 tap columns][2 halves][208 rows][16 bytes]
    float* dks = reinterpret_cast<float*>(btab + B_BYTES);                  // [9 taps][16 channels]
    int* prog = reinterpret_cast<int*>(dks + 9 * CG);                       // output rows the epilogue has finished
    int* aborted = prog + 1;
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(prog + 2);
    u64* bars = reinterpret_cast<u64*>(btab + B_BYTES + 1024);
    const uint32_t rowfull0 = smem_u32(bars), rowdone0 = rowfull0 + 8 * NRING, accfull0 = rowdone0 + 8 * NRING,
                   cfull0 = accfull0 + 8 * SLOTS;
    unsigned char* cring = smem + kCopyRingOffset;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < NRING; ++s) { mbar_init(rowfull0 + 8 * s, 1); mbar_init(rowdone0 + 8 * s, 1); }
        for (int s = 0; s < SLOTS; ++s) mbar_init(accfull0 + 8 * s, 1);
        for (int s = 0; s < kCopySlots; ++s) mbar_init(cfull0 + 8 * s, 1);
        *prog = 0; *aborted = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {                                        // all 512 columns of this SM's tensor memory (one CTA per SM)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_base_slot;
    if (p.wait_first) pdl_wait_primary();
    pdl_launch_dependents();

    // ---- this CTA's rows: image b, strip sx, rows [ya, yb) -------------------------------------------
    unsigned u = blockIdx.x;
    const int seg = (int)(u % (unsigned)p.segs); u /= (unsigned)p.segs;
    const int sx = (int)(u % (unsigned)p.strips);
    const int b = (int)(u / (unsigned)p.strips);
    const int ya = seg * p.seg_rows, yb = min(p.H, ya + p.seg_rows), L = yb - ya;
    const int x0 = sx * MW;
    const int n_in = L + K13 - 1;                           // input rows ya - 6 .. yb + 5, index n = row - (ya - 6)

    // ---- B operands: btab[j][half][(12 - i) * 16 + n][k % 8] = w_dense[n][half * 8 + k % 8][i][j] ------------
    // The weights are gathered with a stride of 169 elements.  From global memory that is 28 rounds of dependent
    // 2-byte loads per thread; instead half of w_dense at a time (8 output channels, 43 KB) is copied, coalesced,
    // into the still empty input ring and the rows are gathered from there.
    {
        uint4* bt = reinterpret_cast<uint4*>(btab);
        constexpr int HALF_W = 8 * CG * K13 * K13;                              // elements of 8 output channels
        static_assert(HALF_W * 2 <= NRING * ROW_BYTES && (HALF_W * 2) % 16 == 0, "staging fits the ring");
        for (int nh = 0; nh < 2; ++nh) {
            const unsigned short* w;
            if (p.w_aligned) {
                const uint4* src = reinterpret_cast<const uint4*>(p.w_dense + (size_t)nh * HALF_W);
                uint4* dst = reinterpret_cast<uint4*>(ring);
                for (int e = tid; e < HALF_W * 2 / 16; e += kThreads) dst[e] = __ldg(src + e);
                __syncthreads();
                w = reinterpret_cast<const unsigned short*>(ring);
            } else {
                w = reinterpret_cast<const unsigned short*>(p.w_dense) + (size_t)nh * HALF_W;
            }
            for (int e = tid; e < K13 * 2 * NBLK * 8; e += kThreads) {           // one 16-byte row each: (j, half, i, n % 8)
                const int n8 = e & 7, ii = (e >> 3) % NBLK, h = ((e >> 3) / NBLK) & 1, j = (e >> 3) / (2 * NBLK);
                const int i = (K13 - 1) - ii;
                unsigned v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) v[q] = w[((size_t)(n8 * CG + h * 8 + q) * K13 + i) * K13 + j];
                bt[(j * 2 + h) * (NBLK * CG) + ii * CG + nh * 8 + n8] =
                    make_uint4(v[0] | (v[1] << 16), v[2] | (v[3] << 16), v[4] | (v[5] << 16), v[6] | (v[7] << 16));
            }
            __syncthreads();                                                     // the staging area is re-used
        }
    }
    // clear the accumulators: every instruction accumulates, a row's columns are cleared again after it is read
    if (warp >= 2) {
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        for (int s = 0; s < SLOTS; ++s) tmem_zero16(lane_base + (uint32_t)(s * CG));
        tmem_wait_st();
    }
    fence_async_smem();                                     // the B table is read through the async proxy
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (warp == 0) {
        // ======================= input rows by TMA ====================================================
        if (lane == 0) {
            bool alive = true;
            for (int n = 0; n < n_in && alive; ++n) {
                const int slot = n % NRING;
                if (n >= NRING) {
                    // the slot's previous row (n - 16) must have been consumed by the tensor cores and, if the 3x3
                    // part of an output row reads it (rows n - 21 .. of this CTA's range), by the epilogue
                    alive = mbar_wait(rowdone0 + 8 * slot, (unsigned)(((n - NRING) / NRING) & 1), p.ctrl, 0xD0000000u | (unsigned)n);
                    const int need = min(n - 20, L);
                    unsigned polls = 0;
                    while (alive && ld_acquire_cta(prog) < need) {
                        __nanosleep(64);
                        if (++polls > kPollLimit || ld_acquire_cta(aborted)) alive = false;
                    }
                    if (!alive) { if (p.ctrl) { atomicExch(p.ctrl, kDevTimeout); atomicExch(p.ctrl + 1, 0xD1000000u | (unsigned)n); } st_release_cta(aborted, 1); break; }
                }
                const uint32_t dst = smem_u32(ring + (size_t)slot * ROW_BYTES), bar = rowfull0 + 8 * slot;
                mbar_expect_tx(bar, ROW_BYTES);
                tma_load_4d(dst, &map_half, bar, 0, x0 - P6, ya - P6 + n, b);
            }
        }
    } else if (warp == 1) {
        // ======================= tensor-core instructions =============================================
        if (lane == 0) {
            bool alive = true;
            const uint32_t ring_a = smem_u32(ring), btab_a = smem_u32(btab);
            for (int n = 0; n < n_in && alive; ++n) {
                const int slot = n % NRING;
                alive = mbar_wait(rowfull0 + 8 * slot, (unsigned)((n / NRING) & 1), p.ctrl, 0xD2000000u | (unsigned)n);
                // the columns of the output row this input row opens (n, if it exists) were cleared by the epilogue of row n - 32
                if (n >= SLOTS && n < L) {
                    unsigned polls = 0;
                    while (alive && ld_acquire_cta(prog) < n - SLOTS + 1) {
                        __nanosleep(64);
                        if (++polls > kPollLimit || ld_acquire_cta(aborted)) alive = false;
                    }
                }
                if (!alive) { if (p.ctrl) { atomicExch(p.ctrl, kDevTimeout); atomicExch(p.ctrl + 1, 0xD3000000u | (unsigned)n); } st_release_cta(aborted, 1); break; }
                tc_fence_after();
                // input row n feeds output rows n - 12 + c, c = 0 .. 12 (kernel row 12 - c), those inside [0, L)
                const int c_lo = max(0, (K13 - 1) - n), c_hi = min(K13 - 1, L - 1 - n + (K13 - 1));
                if (c_lo <= c_hi) {
                    const int cnt = c_hi - c_lo + 1, s0 = (n - (K13 - 1) + c_lo) % SLOTS;
                    const int cnt1 = min(cnt, SLOTS - s0), cnt2 = cnt - cnt1;      // the row slots wrap around at 32
                    for (int j = 0; j < K13; ++j) {
                        const unsigned long long da = smem_desc_sw32(ring_a + (uint32_t)(slot * ROW_BYTES + 32 * j));
                        const uint32_t bj = btab_a + (uint32_t)(j * BJ_BYTES + c_lo * CG * 16);
                        mma_f16(tmem + (uint32_t)(s0 * CG), da, smem_desc(bj, BHALF_BYTES, 128), instr_desc(cnt1 * CG));
                        if (cnt2 > 0)
                            mma_f16(tmem, da, smem_desc(bj + (uint32_t)(cnt1 * CG * 16), BHALF_BYTES, 128), instr_desc(cnt2 * CG));
                    }
                }
                mma_commit(rowdone0 + 8 * slot);                           // arrives when the instructions above have read the row
                if (n >= K13 - 1) mma_commit(accfull0 + 8 * ((n - (K13 - 1)) % SLOTS));   // output row n - 12 is complete
            }
        }
    } else if (warp == 6) {
        // ======================= copy-through of the identity channels: TMA in, TMA out ================
        // this CTA's rows of its strip, a strip row (or a part of it) per chunk, through a ring of two slots
        if (lane == 0 && p.copy_cc != 0) {
            bool alive = true;
            const int per_row = MW / p.copy_pw, chunks = L * per_row;
            const unsigned bytes = (unsigned)(p.copy_cc * p.copy_pw * 2);
            auto coords = [&](int ch, int& cx, int& cy) { cy = ya + ch / per_row; cx = x0 + (ch % per_row) * p.copy_pw; };
            auto issue = [&](int ch) {
                int cx, cy; coords(ch, cx, cy);
                const int slot = ch % kCopySlots;
                mbar_expect_tx(cfull0 + 8 * slot, bytes);
                tma_load_4d(smem_u32(cring + slot * kCopySlotBytes), &map_cin, cfull0 + 8 * slot, CG, cx, cy, b);
            };
            // chunks wholly outside the image (right of W) are skipped by both cursors alike
            auto inside = [&](int ch) { int cx, cy; coords(ch, cx, cy); return cx < p.W; };
            int next = 0;
            while (next < chunks && !inside(next)) ++next;
            if (next < chunks) issue(next);
            int cur = next;
            while (cur < chunks) {
                int nx = cur + 1;
                while (nx < chunks && !inside(nx)) ++nx;
                if (nx < chunks) {
                    bulk_wait_read<0>();                                    // the store that last used the other slot has read it
                    issue(nx);
                }
                if (alive) alive = mbar_wait(cfull0 + 8 * (cur % kCopySlots), (unsigned)((cur / kCopySlots) & 1), p.ctrl, 0xD6000000u | (unsigned)cur);
                int cx, cy; coords(cur, cx, cy);
                tma_store_4d(&map_cout, smem_u32(cring + (cur % kCopySlots) * kCopySlotBytes), CG, cx, cy, b);
                bulk_commit();
                cur = nx;
            }
            bulk_wait_all<0>();
        }
    } else {
        // ======================= epilogue: one pixel per thread =======================================
        const int et = tid - 64, m = ((warp & 3) * 32) + lane;              // tensor-memory lane = pixel of the strip row
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        if (!p.wait_first) pdl_wait_primary();                               // dk comes from the kernel before this one
        for (int e = et; e < 9 * CG; e += kEpiThreads) dks[e] = __ldcg(p.dk + ((size_t)b * CG + (e % CG)) * 9 + e / CG);
        asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
        bool alive = true;
        const int x = x0 + m;
        for (int yr = 0; yr < L; ++yr) {
            const int slot = yr % SLOTS;
            // one lane asks (a wait that all 32 lanes execute costs the warp over a hundred cycles)
            if (lane == 0 && alive) alive = mbar_wait(accfull0 + 8 * slot, (unsigned)((yr / SLOTS) & 1), p.ctrl, 0xD4000000u | (unsigned)yr);
            if (lane == 0 && !alive) st_release_cta(aborted, 1);
            __syncwarp();
            tc_fence_after();
            uint32_t r[16];
            tmem_ld16(lane_base + (uint32_t)(slot * CG), r);
            tmem_zero16(lane_base + (uint32_t)(slot * CG));
            float acc[CG];
#pragma unroll
            for (int c = 0; c < CG; ++c) acc[c] = __uint_as_float(r[c]);
            // dynamic 3x3 kernel, depth-wise, fp32 (Eq. 4 line 3, second term): input rows yr + 5 .. yr + 7 of the ring,
            // pixels m + 5 .. m + 7 of the staged row
#pragma unroll
            for (int a = 0; a < 3; ++a) {
                const int rslot = (yr + 5 + a) % NRING;
                const unsigned char* rowp = ring + (size_t)rslot * ROW_BYTES;
#pragma unroll
                for (int bb = 0; bb < 3; ++bb) {
                    // the pixel's two 16-byte halves are swapped where bit 7 of its address is set (32-byte swizzle)
                    const int px = m + 5 + bb, sw = ((rslot * (ROW_BYTES / 128) + (px >> 2)) & 1) * 16;
                    const uint4 lo = *reinterpret_cast<const uint4*>(rowp + (size_t)px * 32 + sw);
                    const uint4 hi = *reinterpret_cast<const uint4*>(rowp + (size_t)px * 32 + (16 - sw));
                    float f[16];
                    unpack16<__nv_bfloat16>(lo, f);
                    unpack16<__nv_bfloat16>(hi, f + 8);
                    const float4* d4 = reinterpret_cast<const float4*>(dks + (a * 3 + bb) * CG);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float4 d = d4[q];
                        acc[4 * q] = fmaf(d.x, f[4 * q], acc[4 * q]);
                        acc[4 * q + 1] = fmaf(d.y, f[4 * q + 1], acc[4 * q + 1]);
                        acc[4 * q + 2] = fmaf(d.z, f[4 * q + 2], acc[4 * q + 2]);
                        acc[4 * q + 3] = fmaf(d.w, f[4 * q + 3], acc[4 * q + 3]);
                    }
                }
            }
            if (x < p.W) {
                uint32_t o[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const __nv_bfloat162 h2 = __floats2bfloat162_rn(acc[2 * q], acc[2 * q + 1]);
                    o[q] = *reinterpret_cast<const uint32_t*>(&h2);
                }
                uint4* dst = reinterpret_cast<uint4*>(p.out + (((size_t)b * p.H + ya + yr) * p.W + x) * p.C);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            }
            tmem_wait_st();                                                   // the row's columns are cleared
            tc_fence_before();
            asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
            if (et == 0) st_release_cta(prog, yr + 1);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// ---- host side ------------------------------------------------------------------------------------
// [B][H][W][C] bf16 as a 4-D map {C, W, H, B} with a box of 8 channels x SPX pixels x 1 row.
inline int try_launch_dense_umma(int B, int C, int Ca, int H, int W, int K, int dtype, int layout, const void* x,
                                 const void* w_dense, const float* dk, void* out, unsigned* ctrl, cudaStream_t st,
                                 bool dependent, int* launches, std::string* err) {
    if (K != K13 || dtype != 1 /*bf16*/ || layout != kNHWC || Ca != CG || C % 8 != 0) return kNotApplicable;
    if ((reinterpret_cast<uintptr_t>(w_dense) & 1) != 0) return kNotApplicable;
    const int sms = sm_count();
    if (sms <= 0) return kNotApplicable;
    Params p;
    p.B = B; p.C = C; p.H = H; p.W = W;
    p.strips = (W + MW - 1) / MW;
    // row ranges: about one CTA per SM, at least 8 rows each (12 more are read above and below a range)
    long long want = (long long)sms / ((long long)B * p.strips);
    if (want < 1) want = 1;
    int rows = (int)((H + want - 1) / want);
    if (rows < 8) rows = H < 8 ? H : 8;
    p.seg_rows = rows;
    p.segs = (H + rows - 1) / rows;
    const long long ctas = (long long)B * p.strips * p.segs;
    if (ctas > 0x3fffffffLL) return kNotApplicable;
    p.w_dense = static_cast<const __nv_bfloat16*>(w_dense);
    p.dk = dk; p.out = static_cast<__nv_bfloat16*>(out); p.ctrl = ctrl;
    p.wait_first = dependent ? 0 : 1;
    p.w_aligned = (reinterpret_cast<uintptr_t>(w_dense) & 15) == 0 ? 1 : 0;
    const int cc = C - Ca;
    p.copy_cc = cc; p.copy_pw = 0;
    if (cc > 256) return kNotApplicable;
    if (cc > 0) {
        int pw = MW;
        while (pw > 8 && cc * 2 * pw > kCopySlotBytes) pw >>= 1;
        if (cc * 2 * pw > kCopySlotBytes) return kNotApplicable;
        p.copy_pw = pw;
    }
    CUtensorMap m_half, m_cin, m_cout;
    {   // one staged row per load: 16 channels x SPX pixels, written with the 32-byte swizzle the A descriptor names
        EncodeTiledFn fn = encode_fn();
        if (!fn) return kNotApplicable;
        const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
        const cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
        const cuuint32_t box[4] = {(cuuint32_t)CG, (cuuint32_t)SPX, 1, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (fn(&m_half, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_64B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return kNotApplicable;
    }
    if (cc > 0) {
        if (!make_map(&m_cin, x, B, C, H, W, cc, p.copy_pw, 1)) return kNotApplicable;
        if (!make_map(&m_cout, out, B, C, H, W, cc, p.copy_pw, 1)) return kNotApplicable;
    } else {
        m_cin = m_half; m_cout = m_half;
    }
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return kNotApplicable;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(stencil_dense_umma_nhwc_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return kNotApplicable; }
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, stencil_dense_umma_nhwc_bf16, m_half, m_cin, m_cout, p);
    if (e != cudaSuccess) {
        char buf[256];
        snprintf(buf, sizeof buf, "stencil_dense_umma_nhwc_bf16 launch: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e));
        *err = buf;
        return 7;  // ESC_ERR_CUDA
    }
    ++*launches;
    return 0;
}

}}}  // namespace esc::tma::umma

// C ABI of the ConvAttn forward library: argument checks, scratch layout, kernel selection and
// launches.  The arithmetic lives in the kernels (gap_dynkernel.cuh, stencil_generic.cuh,
// stencil_tma.cuh); nothing here touches tensor data on the host.
#include "../../include/esc_convattn.h"

#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <utility>

#include "common.cuh"
#include "gap_dynkernel.cuh"
#include "stencil_generic.cuh"
#include "stencil_tma.cuh"
#include "stencil_toeplitz.cuh"
#include "stencil_toeplitz_nchw.cuh"
#include "backward_toeplitz.cuh"
#include "backward_toeplitz_nchw.cuh"
#include "stencil_dense.cuh"
#include "stencil_dense_umma.cuh"
#include <type_traits>
#include "backward.cuh"
#include "backward_pw.cuh"
#include "backward_dense.cuh"
#include "conv_fuse.cuh"
#include "conv_fuse_backward.cuh"

namespace {

thread_local std::string g_last_error;
thread_local int g_last_path = 0;
thread_local int g_last_tile_w = 0;
thread_local int g_tile_policy = 0;      // 0 = by cost, else the tile width to use
thread_local int g_engine_policy = 0;    // ESC_ENGINE_AUTO / _FP32 / _TENSOR for the depth-wise stencil
thread_local int g_last_launches = 0;
thread_local int g_dense_engine = 0;     // 0: tcgen05 kernel where it applies, 1: the mma.sync kernel
thread_local bool g_fuse_stage1 = true;  // tensor-core kernel: stage 1 inside it where every CTA has at most two units

int cuda_fail(cudaError_t e, const char* what) {
    char buf[320];
    snprintf(buf, sizeof buf, "%s: %s (%s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
    g_last_error = buf;
    return ESC_ERR_CUDA;
}
#define ESC_CUDA(call)                                        \
    do {                                                      \
        cudaError_t e__ = (call);                             \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
    } while (0)

size_t elem_size(int dtype) { return dtype == ESC_BF16 ? 2 : 4; }

struct Problem {
    int B, C, Ca, H, W, K, dtype, layout;
    const void* w_point = nullptr;   // [Ca][Ca] point-wise filter LK^c of the decomposed form (Eq. 5), or none
    bool dense = false;              // w_large is the dense kernel [Ca][Ca][K][K] of Section 3.2
    const float* bias = nullptr;     // [B][Ca] constant per (image, channel) added to the attention outputs (backward pass)
    bool skip_copy = false;          // the identity channels are not written (the fused 1x1 convolution reads them from x)
    size_t es() const { return elem_size(dtype); }
    size_t elems() const { return (size_t)B * C * H * W; }
};

int check_shape(const Problem& p) {
    if (p.B <= 0 || p.C <= 0 || p.H <= 0 || p.W <= 0 || p.Ca <= 0 || p.Ca > p.C) return ESC_ERR_SHAPE;
    if (p.K < 3 || (p.K & 1) == 0) return ESC_ERR_SHAPE;   // the 3x3 dynamic kernel is folded into the K x K one
    if (p.K > ESC_MAX_K) return ESC_ERR_UNSUPPORTED;
    if (p.dtype != ESC_F32 && p.dtype != ESC_BF16) return ESC_ERR_UNSUPPORTED;
    if (p.layout != ESC_NCHW && p.layout != ESC_NHWC) return ESC_ERR_UNSUPPORTED;
    // every byte offset the kernels form must fit in 62 bits
    const long double n = (long double)p.B * p.C * p.H * p.W;
    if (n > 1.0e18L) return ESC_ERR_SHAPE;
    return ESC_OK;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_tensors(const Problem& p, const void* x, const void* out) {
    if (!x || !out) return ESC_ERR_NULL;
    if (!aligned(x, 16) || !aligned(out, 16)) return ESC_ERR_ALIGN;
    const uintptr_t xa = reinterpret_cast<uintptr_t>(x), oa = reinterpret_cast<uintptr_t>(out);
    const size_t bytes = p.elems() * p.es();
    if (xa < oa + bytes && oa < xa + bytes) return ESC_ERR_ALIAS;
    return ESC_OK;
}

// ---- workspace layout -------------------------------------------------------------------
//   [ctrl words: header + B arrival counters + B launch flags][pad to 256][dk: B*Ca*9 floats][pad]
//   [partials: B*S*Ca floats][pad][per-unit sums of the one-launch form: kMaxFusedUnits * SMs * 16 floats][pad]
//   [large kernel padded to 13 x 13]
size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Workspace {
    unsigned* ctrl;
    unsigned* arrivals;
    unsigned* flags;
    float* dk;
    float* partial;
    float* unit_sums;
    void* lk_pad;                    // [Ca][13][13] elements: a smaller large kernel zero-padded for the tensor-core kernels
};

bool is_large_map(int B, long long HW) { return (long double)B * HW >= 1.5e6L; }

// SM count of the current device; a B200's 148 where no device can be asked (size queries on a
// machine without a GPU).
int sms_or_nominal() {
    const int v = esc::tma::sm_count();
    return v > 0 ? v : 148;
}

// Grid policy of the GAP kernel.  Narrow: at most one block per SM, which is what fits beside a CTA of the
// FP32 stencil kernel (58 k registers).  Wide: three blocks per SM -- for maps so large that the stencil
// kernel takes many waves and the GAP kernel runs ahead of it rather than beside it, and for batches in
// front of the tensor-core stencil kernel, whose CTAs need every image's dk early (measured on 64 patches
// of 64x64: 35.5 us per forward against 37.8; a single 640x360 map: 37.4 against 36.2, so single images
// keep the narrow grid).
bool wide_gap(int B, long long HW, bool tensor_stencil) {
    return (tensor_stencil && B > 1) || is_large_map(B, HW);
}

int slabs_for(int B, long long HW, bool wide) {
    // At most one work item per block over the whole batch, so that every block walks one item and no
    // image waits for a second round; at least 512 pixels per slab.
    const long long sms = sms_or_nominal();
    const long long target = wide ? 3 * sms : sms;
    long long s = target / B;
    const long long cap = (HW + 511) / 512;
    if (s > cap) s = cap;
    if (s > esc::kMaxSlabs) s = esc::kMaxSlabs;
    if (s < 1) s = 1;
    return (int)s;
}

size_t workspace_bytes(int B, int Ca, long long HW) {
    const int S = slabs_for(B, HW, true);                   // room for either grid policy
    size_t off = round_up((size_t)(esc::kCtrlHeaderWords + 2 * (size_t)B) * 4, 256);
    off += round_up((size_t)B * Ca * 9 * 4, 256);
    off += round_up((size_t)B * S * Ca * 4, 256);
    off += round_up((size_t)esc::tma::toep::kMaxFusedUnits * sms_or_nominal() * 16 * 4, 256);   // unit sums of the one-launch form
    off += round_up((size_t)Ca * 169 * 4, 256);            // padded large kernel
    return off;
}

Workspace carve(void* ws, int B, int Ca, long long HW) {
    Workspace w;
    char* p = static_cast<char*>(ws);
    w.ctrl = reinterpret_cast<unsigned*>(p);
    w.arrivals = w.ctrl + esc::kCtrlHeaderWords;
    w.flags = w.arrivals + B;
    p += round_up((size_t)(esc::kCtrlHeaderWords + 2 * (size_t)B) * 4, 256);
    w.dk = reinterpret_cast<float*>(p);
    p += round_up((size_t)B * Ca * 9 * 4, 256);
    w.partial = reinterpret_cast<float*>(p);
    p += round_up((size_t)B * slabs_for(B, HW, true) * Ca * 4, 256);
    w.unit_sums = reinterpret_cast<float*>(p);
    p += round_up((size_t)esc::tma::toep::kMaxFusedUnits * sms_or_nominal() * 16 * 4, 256);
    w.lk_pad = p;
    return w;
}

int check_workspace(const Problem& p, const void* ws, size_t bytes) {
    if (!ws || !aligned(ws, 256)) return ESC_ERR_WORKSPACE;
    if (bytes < workspace_bytes(p.B, p.Ca, (long long)p.H * p.W)) return ESC_ERR_WORKSPACE;
    return ESC_OK;
}

// ---- stage 1 ------------------------------------------------------------------------------
// The estimator's weights: one linear layer (hidden == 0: w_last [9*Ca][Ca]) or two layers with the
// GELU between them (w_down [hidden][Ca], b_down [hidden], w_last = w_up [9*Ca][hidden]).
struct Estimator {
    const void *w_last, *b_last, *w_down, *b_down;
    int hidden;
};

template <typename T, int LAYOUT>
int launch_gap_t(const Problem& p, const void* x, const Estimator& est,
                 const Workspace& w, float* dk_out, cudaStream_t st, bool wide) {
    const int S = slabs_for(p.B, (long long)p.H * p.W, wide);
    const int sms = sms_or_nominal();
    const long long items = (long long)p.B * S;
    const long long cap = wide ? 3LL * sms : sms;
    const unsigned grid = (unsigned)(items < cap ? items : cap);
    const size_t scratch = (size_t)esc::gap_scratch_floats(LAYOUT, p.C, p.Ca, esc::Elem<T>::kVec);
    const size_t smem = (scratch + p.Ca) * sizeof(float);
    if (smem > 48 * 1024) return ESC_ERR_UNSUPPORTED;
    // Same shared-memory carve-out as the stencil kernel: an SM changes its L1/shared split only
    // when idle, so with different preferences the two kernels could never share an SM.
    static bool carveout_set[esc::tma::kMaxDevices] = {};   // per device and per instantiation
    const int dev = esc::tma::current_device();
    if (dev < 0) return ESC_ERR_UNSUPPORTED;
    if (!carveout_set[dev]) {
        ESC_CUDA(cudaFuncSetAttribute(esc::gap_dynkernel<T, LAYOUT>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                      cudaSharedmemCarveoutMaxShared));
        carveout_set[dev] = true;
    }
    esc::gap_dynkernel<T, LAYOUT><<<grid, esc::kGapThreads, smem, st>>>(
        static_cast<const T*>(x), p.B, p.C, p.Ca, p.H, p.W, S, static_cast<const T*>(est.w_last),
        static_cast<const T*>(est.b_last), static_cast<const T*>(est.w_down), static_cast<const T*>(est.b_down),
        est.hidden, w.partial, w.arrivals, dk_out);
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    return ESC_OK;
}

int launch_gap(const Problem& p, const void* x, const Estimator& est,
               const Workspace& w, float* dk_out, cudaStream_t st, bool tensor_stencil = false) {
    if ((long long)p.B * esc::kMaxSlabs > 0x7fffffffLL) return ESC_ERR_UNSUPPORTED;
    const bool wide = wide_gap(p.B, (long long)p.H * p.W, tensor_stencil);
    if (p.dtype == ESC_F32)
        return p.layout == ESC_NCHW ? launch_gap_t<float, esc::kNCHW>(p, x, est, w, dk_out, st, wide)
                                    : launch_gap_t<float, esc::kNHWC>(p, x, est, w, dk_out, st, wide);
    return p.layout == ESC_NCHW ? launch_gap_t<__nv_bfloat16, esc::kNCHW>(p, x, est, w, dk_out, st, wide)
                                : launch_gap_t<__nv_bfloat16, esc::kNHWC>(p, x, est, w, dk_out, st, wide);
}

int check_estimator(const Problem& p, const Estimator& e) {
    if (!e.w_last || !e.b_last) return ESC_ERR_NULL;
    if (!aligned(e.w_last, p.es()) || !aligned(e.b_last, p.es())) return ESC_ERR_ALIGN;
    if (e.hidden == 0) return ESC_OK;
    if (e.hidden < 0 || e.hidden > esc::kMaxHidden) return ESC_ERR_SHAPE;
    if (!e.w_down || !e.b_down) return ESC_ERR_NULL;
    if (!aligned(e.w_down, p.es()) || !aligned(e.b_down, p.es())) return ESC_ERR_ALIGN;
    return ESC_OK;
}

// ---- stage 2 ------------------------------------------------------------------------------
template <typename U>
int launch_copy_u(const void* x, void* out, long long rows, long long row_b, long long stride_b,
                  long long off_b, cudaStream_t st) {
    const long long u = sizeof(U);
    const long long total = rows * (row_b / u);
    if (total == 0) return ESC_OK;
    long long blocks = (total + 255) / 256;
    if (blocks > 16LL * sms_or_nominal()) blocks = 16LL * sms_or_nominal();
    esc::copy_through<U><<<(unsigned)blocks, 256, 0, st>>>(static_cast<const U*>(x), static_cast<U*>(out), rows,
                                                          row_b / u, stride_b / u, off_b / u);
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    return ESC_OK;
}

int launch_copy(const Problem& p, const void* x, void* out, cudaStream_t st) {
    if (p.Ca == p.C) return ESC_OK;
    const long long es = (long long)p.es(), HW = (long long)p.H * p.W;
    long long rows, row_b, stride_b, off_b;
    if (p.layout == ESC_NCHW) { rows = p.B; row_b = (p.C - p.Ca) * HW * es; stride_b = p.C * HW * es; off_b = p.Ca * HW * es; }
    else { rows = (long long)p.B * HW; row_b = (p.C - p.Ca) * es; stride_b = p.C * es; off_b = p.Ca * es; }
    if (row_b % 16 == 0 && stride_b % 16 == 0 && off_b % 16 == 0) return launch_copy_u<uint4>(x, out, rows, row_b, stride_b, off_b, st);
    if (row_b % 4 == 0 && stride_b % 4 == 0 && off_b % 4 == 0) return launch_copy_u<uint32_t>(x, out, rows, row_b, stride_b, off_b, st);
    return launch_copy_u<uint16_t>(x, out, rows, row_b, stride_b, off_b, st);
}

// The identity channels as a copy job for extra blocks of a stencil launch (blocks == 0: nothing to copy).
esc::CopyJob make_copy_job(const Problem& p, const void* x, void* out, long long first_block, int threads) {
    esc::CopyJob j = {};
    if (p.Ca == p.C) return j;
    const long long es = (long long)p.es(), HW = (long long)p.H * p.W;
    long long rows, row_b, stride_b, off_b;
    if (p.layout == ESC_NCHW) { rows = p.B; row_b = (p.C - p.Ca) * HW * es; stride_b = p.C * HW * es; off_b = p.Ca * HW * es; }
    else { rows = (long long)p.B * HW; row_b = (p.C - p.Ca) * es; stride_b = p.C * es; off_b = p.Ca * es; }
    const int u = (row_b % 16 == 0 && stride_b % 16 == 0 && off_b % 16 == 0) ? 16
                : (row_b % 4 == 0 && stride_b % 4 == 0 && off_b % 4 == 0) ? 4 : 2;
    j.src = x; j.dst = out;
    j.rows = rows; j.row_units = row_b / u; j.stride_units = stride_b / u; j.offset_units = off_b / u;
    j.unit_bytes = u;
    const long long total = rows * j.row_units;
    long long blocks = (total + (long long)threads * 4 - 1) / ((long long)threads * 4);   // about four units per thread
    if (blocks > 8LL * sms_or_nominal()) blocks = 8LL * sms_or_nominal();
    if (blocks < 1) blocks = 1;
    j.first_block = (unsigned)first_block;
    j.blocks = (unsigned)blocks;
    return j;
}

template <typename T, int LAYOUT>
int launch_generic_t(const Problem& p, const void* x, const void* w_large, const float* dk, void* out,
                     cudaStream_t st, bool dependent) {
    const bool regtile = p.K == esc::kRtK;             // the paper's kernel size: a patch of outputs per thread
    // small launches: smaller tiles, more blocks, so that every SM has several
    auto blocks_of = [&](int tx, int ty) { return (long long)p.B * p.Ca * ((p.W + tx - 1) / tx) * ((p.H + ty - 1) / ty); };
    const bool small = regtile && blocks_of(esc::kRtTX, esc::kRtTY) < 4LL * sms_or_nominal();
    const bool tiny = small && blocks_of(esc::RtSmall::TX, esc::RtSmall::TY) < 2LL * sms_or_nominal();
    const int TX = regtile ? (tiny ? esc::RtTiny::TX : small ? esc::RtSmall::TX : esc::kRtTX) : esc::kGenTX;
    const int TY = regtile ? (tiny ? esc::RtTiny::TY : small ? esc::RtSmall::TY : esc::kRtTY) : esc::kGenTY;
    const int tiles_x = (p.W + TX - 1) / TX, tiles_y = (p.H + TY - 1) / TY;
    const long long blocks = (long long)p.B * p.Ca * tiles_x * tiles_y;
    const esc::CopyJob job = make_copy_job(p, x, out, blocks, regtile ? esc::kRtThreads : esc::kGenTX * esc::kGenTY);
    if (blocks + job.blocks > 0x7fffffffLL) return ESC_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(blocks + job.blocks));   // the copy blocks come last
    cfg.blockDim = regtile ? dim3(esc::kRtThreads) : dim3(esc::kGenTX, esc::kGenTY);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    if (regtile && tiny)
        ESC_CUDA(cudaLaunchKernelEx(&cfg, esc::stencil_k13_regtile<T, LAYOUT, esc::RtTiny>, static_cast<const T*>(x),
                                    static_cast<T*>(out), p.C, p.Ca, p.H, p.W, static_cast<const T*>(w_large), static_cast<const T*>(p.w_point), dk,
                                    tiles_x, tiles_y, job, p.bias));
    else if (regtile && small)
        ESC_CUDA(cudaLaunchKernelEx(&cfg, esc::stencil_k13_regtile<T, LAYOUT, esc::RtSmall>, static_cast<const T*>(x),
                                    static_cast<T*>(out), p.C, p.Ca, p.H, p.W, static_cast<const T*>(w_large), static_cast<const T*>(p.w_point), dk,
                                    tiles_x, tiles_y, job, p.bias));
    else if (regtile)
        ESC_CUDA(cudaLaunchKernelEx(&cfg, esc::stencil_k13_regtile<T, LAYOUT, esc::RtLarge>, static_cast<const T*>(x),
                                    static_cast<T*>(out), p.C, p.Ca, p.H, p.W, static_cast<const T*>(w_large), static_cast<const T*>(p.w_point), dk,
                                    tiles_x, tiles_y, job, p.bias));
    else
        ESC_CUDA(cudaLaunchKernelEx(&cfg, esc::stencil_generic<T, LAYOUT>, static_cast<const T*>(x), static_cast<T*>(out),
                                    p.C, p.Ca, p.H, p.W, p.K, static_cast<const T*>(w_large), static_cast<const T*>(p.w_point), dk, tiles_x, tiles_y, job, p.bias));
    ++g_last_launches;
    return ESC_OK;
}

int launch_generic(const Problem& p, const void* x, const void* w_large, const float* dk, void* out,
                   cudaStream_t st, bool dependent) {
    g_last_path = 1;
    g_last_tile_w = 0;
    int rc;
    if (p.dtype == ESC_F32)
        rc = p.layout == ESC_NCHW ? launch_generic_t<float, esc::kNCHW>(p, x, w_large, dk, out, st, dependent)
                                  : launch_generic_t<float, esc::kNHWC>(p, x, w_large, dk, out, st, dependent);
    else
        rc = p.layout == ESC_NCHW ? launch_generic_t<__nv_bfloat16, esc::kNCHW>(p, x, w_large, dk, out, st, dependent)
                                  : launch_generic_t<__nv_bfloat16, esc::kNHWC>(p, x, w_large, dk, out, st, dependent);
    return rc;                                             // the identity channels went along as copy blocks
}

// The tensor-core depth-wise kernels are built for 13 x 13 taps.  A large kernel of odd size K < 13 is the 13 x 13 one with
// zeros around it -- exactly the same convolution -- so it is written, zero-padded, into the workspace once per call and
// handed to those kernels as a 13 x 13 kernel; every other kernel gets the weights as the caller gave them.
template <typename T>
__global__ void pad_large_kernel(const T* __restrict__ w, int Ca, int K, T* __restrict__ out) {
    const int off = (13 - K) / 2;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < Ca * 169; e += gridDim.x * blockDim.x) {
        const int c = e / 169, i = (e % 169) / 13 - off, j = e % 13 - off;
        out[e] = ((unsigned)i < (unsigned)K && (unsigned)j < (unsigned)K) ? w[((size_t)c * K + i) * K + j] : T(0.0f);
    }
}
struct TensorLk {
    const void* w;
    int K;
};
TensorLk tensor_lk(const Problem& p, const void* x, const void* out, const void* w_large, void* pad, cudaStream_t st) {
    TensorLk t{w_large, p.K};
    if (p.dense || p.dtype != ESC_BF16 || p.K >= esc::tma::K13 || !pad || g_engine_policy == ESC_ENGINE_FP32 || g_tile_policy != 0) return t;
    if (!esc::tma::toep::applies(p.C, p.Ca, esc::tma::K13, p.dtype, p.layout) &&
        !esc::tma::toepn::applies(p.C, p.Ca, p.H, p.W, esc::tma::K13, p.dtype, p.layout, x, out))
        return t;
    pad_large_kernel<__nv_bfloat16><<<(p.Ca * 169 + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(w_large), p.Ca, p.K,
                                                                            static_cast<__nv_bfloat16*>(pad));
    if (cudaGetLastError() != cudaSuccess) return t;
    ++g_last_launches;
    t.w = pad; t.K = esc::tma::K13;
    return t;
}

int launch_stencil(const Problem& p0, const void* x, const void* w_large0, const float* dk, void* out,
                   unsigned* ctrl, cudaStream_t st, bool dependent, const TensorLk* tl = nullptr) {
    // the tensor-core kernels see the (possibly padded) 13 x 13 kernel, everything else the caller's
    Problem p = p0;
    const void* w_large = w_large0;
    if (tl) { p.K = tl->K; w_large = tl->w; }
    // Depth-wise K = 13 on NHWC bf16: the tensor-core (Toeplitz) kernel unless the caller pinned the FP32
    // kernel (by engine or by one of its tile widths) or asked for the point-wise mix, which only the
    // FP32 kernel carries.
    if ((!p.w_point || p.Ca == esc::tma::CG) && g_engine_policy != ESC_ENGINE_FP32 && g_tile_policy == 0) {
        int tw = 0;
        const int rc = esc::tma::toep::try_launch_toeplitz(p.B, p.C, p.Ca, p.H, p.W, p.K, p.dtype, p.layout, x, w_large, dk, p.bias,
                                                           out, ctrl, st, dependent, &g_last_launches, &g_last_error, &tw, p.skip_copy, p.w_point);
        if (rc == ESC_OK) { g_last_path = 4; g_last_tile_w = tw; return ESC_OK; }
        if (rc != esc::tma::kNotApplicable) return rc;
        {                                                    // the same arithmetic on NCHW tensors
            const int rn = esc::tma::toepn::try_launch(p.B, p.C, p.Ca, p.H, p.W, p.K, p.dtype, p.layout, x, w_large, dk, p.bias, out,
                                                       ctrl, st, dependent, &g_last_launches, &g_last_error, p.w_point, p.skip_copy);
            if (rn == ESC_OK) { g_last_path = 6; g_last_tile_w = esc::tma::toepn::TW; return ESC_OK; }
            if (rn != esc::tma::kNotApplicable) return rn;
        }
    }
    if (p.skip_copy) return ESC_ERR_UNSUPPORTED;           // only the tensor-core kernel can leave the identity channels out
    p.K = p0.K; w_large = w_large0;
    if (g_engine_policy == ESC_ENGINE_TENSOR) return launch_generic(p, x, w_large, dk, out, st, dependent);
    int tile_w = g_tile_policy;
    int rc = esc::tma::try_launch(p.B, p.C, p.Ca, p.H, p.W, p.K, p.dtype, p.layout, x, w_large, p.w_point, dk, p.bias, out,
                                  ctrl, st, dependent, &g_last_launches, &g_last_error, &tile_w);
    if (rc == ESC_OK) { g_last_path = 2; g_last_tile_w = tile_w; return ESC_OK; }
    if (rc != esc::tma::kNotApplicable) return rc;
    return launch_generic(p, x, w_large, dk, out, st, dependent);
}

// Whether launch_stencil will take the tensor-core kernel for this problem (same conditions).
bool tensor_stencil_follows(const Problem& p) {
    return !p.dense && (!p.w_point || (p.Ca == esc::tma::CG && !p.bias)) && g_engine_policy != ESC_ENGINE_FP32 && g_tile_policy == 0 &&
           esc::tma::toep::applies(p.C, p.Ca, p.K, p.dtype, p.layout);
}

// ---- library-owned scratch for the entry point that has no workspace argument --------------
struct Scratch { void* ptr = nullptr; size_t bytes = 0; };
std::mutex g_scratch_mu;
std::map<std::pair<int, void*>, Scratch> g_scratch;

int get_scratch(size_t need, cudaStream_t st, void** out) {
    int dev = 0;
    ESC_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    Scratch& s = g_scratch[{dev, (void*)st}];
    if (s.bytes < need) {
        if (s.ptr) { ESC_CUDA(cudaFree(s.ptr)); s.ptr = nullptr; s.bytes = 0; }   // cudaFree waits for pending work
        const size_t cap = round_up(need, 1 << 20);
        ESC_CUDA(cudaMalloc(&s.ptr, cap));
        ESC_CUDA(cudaMemset(s.ptr, 0, cap));
        s.bytes = cap;
    }
    *out = s.ptr;
    return ESC_OK;
}

template <typename T, int LAYOUT>
int launch_dense_generic_t(const Problem& p, const void* x, const void* w_dense, const float* dk, void* out,
                           cudaStream_t st, bool dependent) {
    const long long total = (long long)p.B * p.Ca * p.H * p.W;
    long long blocks = (total + 255) / 256;
    if (blocks > 8LL * sms_or_nominal()) blocks = 8LL * sms_or_nominal();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    ESC_CUDA(cudaLaunchKernelEx(&cfg, esc::tma::stencil_dense_generic<T, LAYOUT>, static_cast<const T*>(x),
                                static_cast<T*>(out), p.B, p.C, p.Ca, p.H, p.W, p.K, static_cast<const T*>(w_dense), dk));
    ++g_last_launches;
    return ESC_OK;
}

// Dense large kernel: tensor-core kernel where it applies, one thread per output elsewhere; the identity
// channels go through the copy kernel either way.
int launch_stencil_dense(const Problem& p, const void* x, const void* w_dense, const float* dk, void* out,
                         unsigned* ctrl, cudaStream_t st, bool dependent) {
    g_last_tile_w = 0;
    if (g_dense_engine == 0) {
        const int urc = esc::tma::umma::try_launch_dense_umma(p.B, p.C, p.Ca, p.H, p.W, p.K, p.dtype, p.layout, x, w_dense, dk, out,
                                                              ctrl, st, dependent, &g_last_launches, &g_last_error);
        if (urc == ESC_OK) { g_last_path = 5; g_last_tile_w = esc::tma::umma::MW; return ESC_OK; }
        if (urc != esc::tma::kNotApplicable) return urc;
    }
    esc::CopyJob job = make_copy_job(p, x, out, 0, esc::tma::dense::kThreads);
    if (job.blocks > (unsigned)sms_or_nominal()) job.blocks = (unsigned)sms_or_nominal();   // every block of that launch takes a whole SM
    int rc = esc::tma::try_launch_dense(p.B, p.C, p.Ca, p.H, p.W, p.K, p.dtype, p.layout, x, w_dense, dk, out, ctrl,
                                        st, dependent, job, &g_last_launches, &g_last_error);
    if (rc == ESC_OK) {
        g_last_path = 3;
        g_last_tile_w = esc::tma::dense::TW;
        return ESC_OK;                                     // the identity channels went along as copy blocks
    } else if (rc == esc::tma::kNotApplicable) {
        g_last_path = 1;
        if (p.dtype == ESC_F32)
            rc = p.layout == ESC_NCHW ? launch_dense_generic_t<float, esc::kNCHW>(p, x, w_dense, dk, out, st, dependent)
                                      : launch_dense_generic_t<float, esc::kNHWC>(p, x, w_dense, dk, out, st, dependent);
        else
            rc = p.layout == ESC_NCHW ? launch_dense_generic_t<__nv_bfloat16, esc::kNCHW>(p, x, w_dense, dk, out, st, dependent)
                                      : launch_dense_generic_t<__nv_bfloat16, esc::kNHWC>(p, x, w_dense, dk, out, st, dependent);
    }
    if (rc != ESC_OK) return rc;
    return launch_copy(p, x, out, st);
}

int forward_impl(const Problem& p0, const void* x, const void* w_large0, const Estimator& est,
                 void* out, void* ws, cudaStream_t st) {
    const Workspace w = carve(ws, p0.B, p0.Ca, (long long)p0.H * p0.W);
    // what the tensor-core kernels see: a smaller large kernel zero-padded to 13 x 13 (launched first, so that the GAP
    // kernel stays the stencil kernel's immediate predecessor)
    const TensorLk tl = tensor_lk(p0, x, out, w_large0, w.lk_pad, st);
    Problem p = p0;
    p.K = tl.K;
    const void* w_large = tl.w;
    // Small problems on the tensor-core kernel: one launch, stage 1 inside the stencil kernel.
    if (g_fuse_stage1 && tensor_stencil_follows(p)) {
        const esc::tma::toep::Fused fu{est.w_last, est.b_last, est.w_down, est.b_down, est.hidden, w.unit_sums, w.arrivals, w.flags};
        int tw = 0;
        const int rc = esc::tma::toep::try_launch_fused(p.B, p.C, p.Ca, p.H, p.W, p.K, p.dtype, p.layout, x, w_large, fu, out,
                                                        w.ctrl, st, &g_last_launches, &g_last_error, &tw, p.skip_copy, p.w_point);
        if (rc == ESC_OK) { g_last_path = 4; g_last_tile_w = tw; return ESC_OK; }
        if (rc != esc::tma::kNotApplicable) {
            // a cooperative launch can be refused (SMs held by another context): fall back to two kernels
            (void)cudaGetLastError();
            g_last_error.clear();
        }
    }
    if (g_fuse_stage1 && !p.dense && (!p.w_point || p.Ca == esc::tma::CG) && !p.bias && g_engine_policy != ESC_ENGINE_FP32 &&
        g_tile_policy == 0) {
        const esc::tma::toep::Fused fu{est.w_last, est.b_last, est.w_down, est.b_down, est.hidden, w.unit_sums, w.arrivals, w.flags};
        const int rc = esc::tma::toepn::try_launch_fused(p.B, p.C, p.Ca, p.H, p.W, p.K, p.dtype, p.layout, x, w_large, fu, out, w.ctrl, st,
                                                         &g_last_launches, &g_last_error, p.w_point, p.skip_copy);
        if (rc == ESC_OK) { g_last_path = 6; g_last_tile_w = esc::tma::toepn::TW; return ESC_OK; }
        if (rc != esc::tma::kNotApplicable) { (void)cudaGetLastError(); g_last_error.clear(); }
    }
    const bool tensor_nchw = !p.dense && (!p.w_point || p.Ca == esc::tma::CG) && !p.bias && g_engine_policy != ESC_ENGINE_FP32 && g_tile_policy == 0 &&
                             esc::tma::toepn::applies(p.C, p.Ca, p.H, p.W, p.K, p.dtype, p.layout, x, out);
    int rc = launch_gap(p0, x, est, w, w.dk, st, tensor_stencil_follows(p) || tensor_nchw);
    if (rc != ESC_OK) return rc;
    if (p0.dense) return launch_stencil_dense(p0, x, w_large0, w.dk, out, w.ctrl, st, /*dependent=*/true);
    return launch_stencil(p0, x, w_large0, w.dk, out, w.ctrl, st, /*dependent=*/true, &tl);
}

// ---- backward pass -------------------------------------------------------------------------
// Workspace: [ctrl 256 B | per-tile partial tap gradients B*Ca*tiles*kSlot | tap gradients B*Ca*kSlot |
//             rotated LK Ca*169 elements | rotated dk B*Ca*9 | constants B*Ca], each part 256-byte aligned.
struct BackwardWs {
    unsigned* ctrl;
    float *part, *gtap, *dk_flip, *bias;
    float *act, *gt;                 // two-layer estimator: activations and g_t, [B][kMaxHidden] each
    void* lk_pad;                    // the rotated large kernel zero-padded to 13 x 13 for the tensor-core kernels
    void* w_flip;
    float *xs_part, *gp_part;        // decomposed form: per-chunk sums of x_att [B][chunks][Ca] and of g_P [B * chunks][Ca * Ca]
    int chunks;                      // chunks of pixels per image in those
    bool patch_xsum;                 // the tap-gradient kernels ran on the mixed features: take the sums of x_att from xs_part
    size_t bytes;
    float* dense_part;               // dense large kernel: the blocks' tap sums [blocks][16][16][169]
    void* wd_flip;                   // the dense kernel with swapped channel axes and rotated taps
    int dense_blocks;
    size_t bytes_dense;              // bytes with those two behind the rest
};
BackwardWs carve_backward(void* ws, const Problem& p) {
    // sized for whichever tiling of the tap-gradient kernels has more tiles (32x32, or 64x16 on the tensor cores)
    const int tiles = std::max(((p.W + esc::bwd::n8::TX - 1) / esc::bwd::n8::TX) * ((p.H + esc::bwd::n8::TY - 1) / esc::bwd::n8::TY),
                               esc::bwd::toep::tiles_of(p.H, p.W));
    BackwardWs w;
    char* base = static_cast<char*>(ws);
    size_t off = 256;
    w.ctrl = reinterpret_cast<unsigned*>(base);
    w.part = reinterpret_cast<float*>(base + off); off += round_up((size_t)p.B * p.Ca * tiles * esc::bwd::kSlot * 4, 256);
    w.gtap = reinterpret_cast<float*>(base + off); off += round_up((size_t)p.B * p.Ca * esc::bwd::kSlot * 4, 256);
    w.w_flip = base + off;                          off += round_up((size_t)p.Ca * esc::bwd::TAPS * 4, 256);
    w.dk_flip = reinterpret_cast<float*>(base + off); off += round_up((size_t)p.B * p.Ca * 9 * 4, 256);
    w.bias = reinterpret_cast<float*>(base + off);  off += round_up((size_t)p.B * p.Ca * 4, 256);
    w.act = reinterpret_cast<float*>(base + off);   off += round_up((size_t)p.B * esc::kMaxHidden * 4, 256);
    w.gt = reinterpret_cast<float*>(base + off);    off += round_up((size_t)p.B * esc::kMaxHidden * 4, 256);
    w.lk_pad = base + off;                          off += round_up((size_t)p.Ca * esc::bwd::TAPS * 4, 256);
    w.chunks = esc::bwd::pw::chunks_of((long long)p.H * p.W);
    w.patch_xsum = false;
    w.xs_part = reinterpret_cast<float*>(base + off); off += round_up((size_t)p.B * w.chunks * p.Ca * 4, 256);
    w.gp_part = reinterpret_cast<float*>(base + off);
    if (esc::bwd::pw::supported(p.Ca)) off += round_up((size_t)p.B * w.chunks * p.Ca * p.Ca * 4, 256);
    w.bytes = off;
    w.dense_blocks = sms_or_nominal();
    w.dense_part = reinterpret_cast<float*>(base + off); off += round_up((size_t)w.dense_blocks * esc::bwd::dense::kPartFloats * 4, 256);
    w.wd_flip = base + off;                              off += round_up((size_t)esc::bwd::dense::CA * esc::bwd::dense::CA * esc::bwd::TAPS * 4, 256);
    w.bytes_dense = off;
    return w;
}

// Weight gradients the caller asked for (fp32, any may be null): of LK, and of the estimator's layers -- last layer
// (W_dyn, b_dyn, or W_up, b_up) and, for the two-layer estimator, W_down, b_down.
struct BackwardGrads {
    float *g_lk, *g_w_last, *g_b_last, *g_w_down, *g_b_down;
};

template <typename T, int LAYOUT>
int backward_t(const Problem& p, const void* x, const void* go, const void* w_large, const Estimator& est,
               const BackwardWs& w, const BackwardGrads& g, cudaStream_t st) {
    // bf16 NHWC with whole groups of 16 channels: the tensor-core kernel (all tap-gradient kernels form the 13 x 13 taps'
    // gradients, whatever the large kernel's size: a smaller one is their middle)
    int tiles_done = 0;
    if (g_engine_policy != ESC_ENGINE_FP32) {
        const int rt = esc::bwd::toep::try_launch(p.B, p.C, p.Ca, p.H, p.W, esc::bwd::K, p.dtype, p.layout, x, go, w.part, w.ctrl, st,
                                                  &g_last_launches, &g_last_error);
        if (rt == ESC_OK) tiles_done = esc::bwd::toep::tiles_of(p.H, p.W);
        else if (rt != esc::tma::kNotApplicable) return rt;
        if (tiles_done == 0) {                               // the same on NCHW tensors
            const int rn = esc::bwd::toepn::try_launch(p.B, p.C, p.Ca, p.H, p.W, esc::bwd::K, p.dtype, p.layout, x, go, w.part, w.ctrl, st,
                                                       &g_last_launches, &g_last_error);
            if (rn == ESC_OK) tiles_done = esc::bwd::toep::tiles_of(p.H, p.W);
            else if (rn != esc::tma::kNotApplicable) return rn;
        }
    }
    // NHWC with whole octets of channels: eight channels per block, 16-byte loads; else a block per channel
    const bool oct = LAYOUT == esc::kNHWC && p.Ca % 8 == 0 && p.C % 8 == 0;
    const int TXs = oct ? esc::bwd::n8::TX : esc::bwd::TX, TYs = oct ? esc::bwd::n8::TY : esc::bwd::TY;
    const int tiles_x = (p.W + TXs - 1) / TXs, tiles_y = (p.H + TYs - 1) / TYs;
    const long long blocks = (long long)p.B * (oct ? p.Ca / 8 : p.Ca) * tiles_x * tiles_y;
    if (blocks > 0x7fffffffLL) return ESC_ERR_UNSUPPORTED;
    if (tiles_done > 0) {
        // done above
    } else if (oct) {
        static bool attr_set[esc::tma::kMaxDevices] = {};
        const int dev = esc::tma::current_device();
        if (dev < 0) return ESC_ERR_UNSUPPORTED;
        if (!attr_set[dev]) {
            ESC_CUDA(cudaFuncSetAttribute(esc::bwd::tap_grad_nhwc8<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)esc::bwd::n8::kSmemBytes));
            attr_set[dev] = true;
        }
        esc::bwd::tap_grad_nhwc8<T><<<(unsigned)blocks, esc::bwd::n8::kThreads, esc::bwd::n8::kSmemBytes, st>>>(
            static_cast<const T*>(x), static_cast<const T*>(go), p.C, p.Ca, p.H, p.W, tiles_x, tiles_y, w.part);
    } else {
        esc::bwd::tap_grad<T, LAYOUT><<<(unsigned)blocks, esc::bwd::kThreads, 0, st>>>(
            static_cast<const T*>(x), static_cast<const T*>(go), p.C, p.Ca, p.H, p.W, tiles_x, tiles_y, w.part);
    }
    ESC_CUDA(cudaGetLastError());
    if (tiles_done == 0) ++g_last_launches;
    esc::bwd::sum_tiles<<<(unsigned)(p.B * p.Ca), esc::bwd::kSumThreads, 0, st>>>(w.part, tiles_done > 0 ? tiles_done : tiles_x * tiles_y, w.gtap);
    ESC_CUDA(cudaGetLastError());
    if (w.patch_xsum) {
        // decomposed form: the sums the tap-gradient kernels took are those of the mixed features; g_W wants the unmixed ones
        const int warps = p.B * p.Ca;
        esc::bwd::pw::sum_x<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(w.xs_part, warps, p.Ca, w.chunks, w.gtap);
        ESC_CUDA(cudaGetLastError());
        ++g_last_launches;
    }
    if (est.hidden == 0) {
        esc::bwd::finish<T><<<esc::bwd::kFinishBlocks, 256, 0, st>>>(w.gtap, p.B, p.Ca, p.H, p.W, p.K, static_cast<const T*>(w_large),
                                                static_cast<const T*>(est.w_last), static_cast<const T*>(est.b_last), g.g_lk,
                                                g.g_w_last, g.g_b_last, static_cast<T*>(w.w_flip), w.dk_flip, w.bias);
        ESC_CUDA(cudaGetLastError());
        g_last_launches += 2;
        return ESC_OK;
    }
    // two-layer estimator: what belongs to one image, then the sums over images
    const size_t smem = (size_t)(10 * p.Ca + 3 * est.hidden) * sizeof(float);
    if (smem > 48 * 1024) return ESC_ERR_UNSUPPORTED;
    esc::bwd::mlp_image<T><<<(unsigned)p.B, 256, smem, st>>>(w.gtap, p.Ca, est.hidden, p.H, p.W, static_cast<const T*>(est.w_down),
                                                             static_cast<const T*>(est.b_down), static_cast<const T*>(est.w_last),
                                                             static_cast<const T*>(est.b_last), w.act, w.gt, w.dk_flip, w.bias);
    ESC_CUDA(cudaGetLastError());
    esc::bwd::mlp_weights<T><<<esc::bwd::kMlpBlocks, 256, 0, st>>>(w.gtap, w.act, w.gt, p.B, p.Ca, est.hidden, p.H, p.W, p.K,
                                                                  static_cast<const T*>(w_large), g.g_lk, g.g_w_down, g.g_b_down,
                                                                  g.g_w_last, g.g_b_last, static_cast<T*>(w.w_flip));
    ESC_CUDA(cudaGetLastError());
    g_last_launches += 3;
    return ESC_OK;
}

// Decomposed form: the two per-pixel kernels around the depth-wise backward pass.
bool pw_vec(const Problem& p) { return p.layout == ESC_NHWC && ((size_t)p.C * p.es()) % 16 == 0 && ((size_t)p.Ca * p.es()) % 16 == 0; }

template <typename T, int LAYOUT, int CA>
int pw_mix_ca(const Problem& p, const void* x, const void* w_point, void* m, const BackwardWs& w, cudaStream_t st) {
    const unsigned blocks = (unsigned)((long long)p.B * w.chunks);
    esc::bwd::pw::mix<T, LAYOUT, CA><<<blocks, esc::bwd::pw::kThreads, 0, st>>>(
        static_cast<const T*>(x), static_cast<const T*>(w_point), static_cast<T*>(m), p.C, (long long)p.H * p.W, w.chunks,
        pw_vec(p) ? 1 : 0, w.xs_part);
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    return ESC_OK;
}
template <typename T, int LAYOUT>
int pw_mix_t(const Problem& p, const void* x, const void* w_point, void* m, const BackwardWs& w, cudaStream_t st) {
    switch (p.Ca) {
        case 4: return pw_mix_ca<T, LAYOUT, 4>(p, x, w_point, m, w, st);
        case 8: return pw_mix_ca<T, LAYOUT, 8>(p, x, w_point, m, w, st);
        case 16: return pw_mix_ca<T, LAYOUT, 16>(p, x, w_point, m, w, st);
        case 32: return pw_mix_ca<T, LAYOUT, 32>(p, x, w_point, m, w, st);
    }
    return ESC_ERR_UNSUPPORTED;
}

template <typename T, int LAYOUT, int CA>
int pw_back_ca(const Problem& p, const void* x, const void* w_point, void* gx, const BackwardWs& w, float* g_wp, cudaStream_t st) {
    constexpr size_t smem = esc::bwd::pw::back_smem_bytes<CA>();
    if (smem > 48 * 1024) {
        static bool attr_set[esc::tma::kMaxDevices] = {};
        const int dev = esc::tma::current_device();
        if (dev < 0) return ESC_ERR_UNSUPPORTED;
        if (!attr_set[dev]) {
            ESC_CUDA(cudaFuncSetAttribute(esc::bwd::pw::back<T, LAYOUT, CA>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            attr_set[dev] = true;
        }
    }
    const unsigned blocks = (unsigned)((long long)p.B * w.chunks);
    esc::bwd::pw::back<T, LAYOUT, CA><<<blocks, esc::bwd::pw::kThreads, smem, st>>>(
        static_cast<const T*>(x), static_cast<const T*>(w_point), static_cast<T*>(gx), w.bias, p.C, (long long)p.H * p.W,
        w.chunks, pw_vec(p) ? 1 : 0, w.gp_part);
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    if (g_wp) {
        const int elems = CA * CA;
        esc::bwd::pw::sum_gp<<<(unsigned)((elems + 7) / 8), 256, 0, st>>>(w.gp_part, elems, (int)blocks, g_wp);
        ESC_CUDA(cudaGetLastError());
        ++g_last_launches;
    }
    return ESC_OK;
}
template <typename T, int LAYOUT>
int pw_back_t(const Problem& p, const void* x, const void* w_point, void* gx, const BackwardWs& w, float* g_wp, cudaStream_t st) {
    switch (p.Ca) {
        case 4: return pw_back_ca<T, LAYOUT, 4>(p, x, w_point, gx, w, g_wp, st);
        case 8: return pw_back_ca<T, LAYOUT, 8>(p, x, w_point, gx, w, g_wp, st);
        case 16: return pw_back_ca<T, LAYOUT, 16>(p, x, w_point, gx, w, g_wp, st);
        case 32: return pw_back_ca<T, LAYOUT, 32>(p, x, w_point, gx, w, g_wp, st);
    }
    return ESC_ERR_UNSUPPORTED;
}

// Dense large kernel: tap gradients of every channel pair, the rotated kernel for the stencil pass, and the constants
// added behind it.
template <typename T, int LAYOUT>
int dense_tap_grad_t(const Problem& p, const void* x, const void* go, const void* w_dense, const BackwardWs& w, float* g_wd,
                     cudaStream_t st) {
    namespace D = esc::bwd::dense;
    static bool attr_set[esc::tma::kMaxDevices] = {};
    const int dev = esc::tma::current_device();
    if (dev < 0) return ESC_ERR_UNSUPPORTED;
    if (!attr_set[dev]) {
        ESC_CUDA(cudaFuncSetAttribute(D::tap_grad_dense<T, LAYOUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)D::kSmemBytes));
        attr_set[dev] = true;
    }
    const int tiles_x = (p.W + D::TX - 1) / D::TX, tiles_y = (p.H + D::TY - 1) / D::TY;
    if (g_wd) {
        if (std::is_same<T, __nv_bfloat16>::value && g_engine_policy != ESC_ENGINE_FP32) {
            // bf16: a matrix product per tap on the tensor cores
            static bool attr_mma[esc::tma::kMaxDevices] = {};
            if (!attr_mma[dev]) {
                ESC_CUDA(cudaFuncSetAttribute(D::mma::tap_grad_dense_bf16<LAYOUT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)D::mma::kSmemBytes));
                attr_mma[dev] = true;
            }
            const int vec = LAYOUT == esc::kNHWC && p.C % 8 == 0 ? 1 : 0;
            const int tiles_ym = (p.H + D::mma::TYM - 1) / D::mma::TYM;
            D::mma::tap_grad_dense_bf16<LAYOUT><<<(unsigned)w.dense_blocks, D::mma::kThreads, D::mma::kSmemBytes, st>>>(
                static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(go), p.B, p.C, p.H, p.W, tiles_x, tiles_ym, vec,
                w.dense_part);
        } else {
            D::tap_grad_dense<T, LAYOUT><<<(unsigned)w.dense_blocks, D::kThreads, D::kSmemBytes, st>>>(
                static_cast<const T*>(x), static_cast<const T*>(go), p.B, p.C, p.H, p.W, tiles_x, tiles_y, w.dense_part);
        }
        ESC_CUDA(cudaGetLastError());
        const int elems = D::CA * D::CA * p.K * p.K;
        D::sum_dense<<<(unsigned)((elems + 255) / 256), 256, 0, st>>>(w.dense_part, w.dense_blocks, p.K, g_wd);
        ESC_CUDA(cudaGetLastError());
        g_last_launches += 2;
    }
    const int elems = D::CA * D::CA * p.K * p.K;
    D::flip_dense<T><<<(unsigned)((elems + 255) / 256), 256, 0, st>>>(static_cast<const T*>(w_dense), p.K, static_cast<T*>(w.wd_flip));
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    return ESC_OK;
}
template <typename T, int LAYOUT>
int dense_add_const_t(const Problem& p, void* gx, const BackwardWs& w, cudaStream_t st) {
    const long long total = (long long)p.B * p.Ca * p.H * p.W;
    long long blocks = (total + 255) / 256;
    if (blocks > 16LL * sms_or_nominal()) blocks = 16LL * sms_or_nominal();
    esc::bwd::dense::add_const<T, LAYOUT><<<(unsigned)blocks, 256, 0, st>>>(static_cast<T*>(gx), w.bias, p.B, p.C, p.Ca, (long long)p.H * p.W);
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    return ESC_OK;
}

// ---- backward pass of Conv_fuse -------------------------------------------------------------------------------
struct FuseBackwardWs {
    void* wt;                        // W_fuse transposed, element type of the tensors
    float* part;                     // [blocks][C * C + C]
    int passes, blocks;
    size_t bytes;
};
FuseBackwardWs carve_fuse_backward(void* ws, int C, long long pixels) {
    FuseBackwardWs w;
    // one block per SM at most (both kernels fill an SM), each with a run of pixels long enough to pay for its final sums
    const long long runs = (pixels + esc::fuse::bwd::kThreads - 1) / esc::fuse::bwd::kThreads, cap = sms_or_nominal();
    w.passes = (int)std::max(2LL, (runs + cap - 1) / cap);
    w.blocks = (int)((runs + w.passes - 1) / w.passes);
    char* base = static_cast<char*>(ws);
    size_t off = 0;
    w.wt = base + off;                              off += round_up((size_t)C * C * 4, 256);
    w.part = reinterpret_cast<float*>(base + off);  off += round_up((size_t)w.blocks * ((size_t)C * C + C) * 4, 256);
    w.bytes = off;
    return w;
}

template <typename T, int LAYOUT, int C>
int fuse_wgrad_c(const void* cat, const void* go, long long HW, long long pixels, const FuseBackwardWs& w, cudaStream_t st) {
    using G = esc::fuse::bwd::Geom<C>;
    if (G::kSmemBytes > 48 * 1024) {
        static bool attr_set[esc::tma::kMaxDevices] = {};
        const int dev = esc::tma::current_device();
        if (dev < 0) return ESC_ERR_UNSUPPORTED;
        if (!attr_set[dev]) {
            ESC_CUDA(cudaFuncSetAttribute(esc::fuse::bwd::wgrad<T, LAYOUT, C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)G::kSmemBytes));
            attr_set[dev] = true;
        }
    }
    esc::fuse::bwd::wgrad<T, LAYOUT, C><<<(unsigned)w.blocks, esc::fuse::bwd::kThreads, G::kSmemBytes, st>>>(
        static_cast<const T*>(cat), static_cast<const T*>(go), HW, pixels, w.passes, w.part);
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    return ESC_OK;
}
template <int C>
int fuse_wgrad_mma_c(const void* cat, const void* go, long long pixels, const FuseBackwardWs& w, cudaStream_t st) {
    namespace M = esc::fuse::bwd::mma;
    static bool attr_set[esc::tma::kMaxDevices] = {};
    const int dev = esc::tma::current_device();
    if (dev < 0) return ESC_ERR_UNSUPPORTED;
    if (!attr_set[dev]) {
        ESC_CUDA(cudaFuncSetAttribute(M::wgrad_bf16_nhwc<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)M::MGeom<C>::kSmemBytes));
        attr_set[dev] = true;
    }
    M::wgrad_bf16_nhwc<C><<<(unsigned)w.blocks, esc::fuse::bwd::kThreads, M::MGeom<C>::kSmemBytes, st>>>(
        static_cast<const __nv_bfloat16*>(cat), static_cast<const __nv_bfloat16*>(go), pixels, w.passes, w.part);
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    return ESC_OK;
}

template <int C>
int fuse_wgrad_mma_nchw_c(const void* cat, const void* go, long long HW, long long pixels, const FuseBackwardWs& w, cudaStream_t st) {
    namespace M = esc::fuse::bwd::mma;
    static bool attr_set[esc::tma::kMaxDevices] = {};
    const int dev = esc::tma::current_device();
    if (dev < 0) return ESC_ERR_UNSUPPORTED;
    if (!attr_set[dev]) {
        ESC_CUDA(cudaFuncSetAttribute(M::wgrad_bf16_nchw<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)M::NGeom<C>::kSmemBytes));
        attr_set[dev] = true;
    }
    M::wgrad_bf16_nchw<C><<<(unsigned)w.blocks, esc::fuse::bwd::kThreads, M::NGeom<C>::kSmemBytes, st>>>(
        static_cast<const __nv_bfloat16*>(cat), static_cast<const __nv_bfloat16*>(go), HW, pixels, w.passes, w.part);
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    return ESC_OK;
}

template <typename T, int LAYOUT>
int fuse_wgrad_t(int C, const void* cat, const void* go, long long HW, long long pixels, const FuseBackwardWs& w, cudaStream_t st) {
    if (std::is_same<T, __nv_bfloat16>::value && LAYOUT == esc::kNCHW && HW % 8 == 0 && g_engine_policy != ESC_ENGINE_FP32) {
        // bf16 NCHW with whole 16-byte pieces per image: the same matrix product, operands without transposition
        switch (C) {
            case 32: return fuse_wgrad_mma_nchw_c<32>(cat, go, HW, pixels, w, st);
            case 48: return fuse_wgrad_mma_nchw_c<48>(cat, go, HW, pixels, w, st);
            case 64: return fuse_wgrad_mma_nchw_c<64>(cat, go, HW, pixels, w, st);
        }
    }
    if (std::is_same<T, __nv_bfloat16>::value && LAYOUT == esc::kNHWC && g_engine_policy != ESC_ENGINE_FP32) {
        // bf16 NHWC: one matrix product over the pixels on the tensor cores
        switch (C) {
            case 32: return fuse_wgrad_mma_c<32>(cat, go, pixels, w, st);
            case 48: return fuse_wgrad_mma_c<48>(cat, go, pixels, w, st);
            case 64: return fuse_wgrad_mma_c<64>(cat, go, pixels, w, st);
        }
    }
    switch (C) {
        case 16: return fuse_wgrad_c<T, LAYOUT, 16>(cat, go, HW, pixels, w, st);
        case 32: return fuse_wgrad_c<T, LAYOUT, 32>(cat, go, HW, pixels, w, st);
        case 48: return fuse_wgrad_c<T, LAYOUT, 48>(cat, go, HW, pixels, w, st);
        case 64: return fuse_wgrad_c<T, LAYOUT, 64>(cat, go, HW, pixels, w, st);
    }
    return ESC_ERR_UNSUPPORTED;
}

// ---- the bounded wait, run on purpose -----------------------------------------------------------------------
// One thread waits, with the kernels' own bounded wait, on a barrier that nothing signals: the wait gives up after its
// poll limit (about a second), records the status and the kernel returns normally.
__global__ void bounded_wait_probe(unsigned* ctrl) {
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x == 0) {
        const uint32_t b = esc::tma::smem_u32(&bar);
        esc::tma::mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        esc::tma::mbar_wait(b, 0, ctrl, 0x5E1F0000u);
    }
}

// ---- fixed scratch for the entry point that must not allocate ------------------------------
// Layout: [kStaticMaxImages arrival counters][kStaticMaxPartials partial sums].  The array lives in
// the library's device image: every GPU that loads the library holds these 64 KiB until exit.
constexpr int kStaticMaxImages = 1024;
constexpr int kStaticMaxPartials = 15360;
static __device__ __align__(256) unsigned g_static_scratch[kStaticMaxImages + kStaticMaxPartials];
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
unsigned* g_static_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device

// In host code `g_static_scratch` is only a handle; the address a kernel can use has to be asked
// for, once per device, with that device current.
int static_scratch_address(unsigned** out) {
    int dev = 0;
    ESC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return ESC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_addr[dev]) {
        void* ptr = nullptr;
        ESC_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        g_static_addr[dev] = static_cast<unsigned*>(ptr);
    }
    *out = g_static_addr[dev];
    return ESC_OK;
}

// ---- host-buffer path ---------------------------------------------------------------------
struct HostPath {
    int dev = -1;
    cudaStream_t st = nullptr;
    void *x = nullptr, *out = nullptr, *wts = nullptr, *ws = nullptr;
    size_t xbytes = 0, wbytes = 0, wsbytes = 0;
};
constexpr int kHostSlots = 2;
std::mutex g_host_mu;
HostPath g_host[kHostSlots];

}  // namespace

extern "C" {

int esc_version(void) { return 120; }

const char* esc_last_error(void) { return g_last_error.c_str(); }

int esc_convattn_last_path(void) { return g_last_path; }
int esc_convattn_last_tile_width(void) { return g_last_tile_w; }
int esc_convattn_set_tile_width(int tile_width) {
    if (tile_width != 0 && tile_width != esc::tma::Geom40::TW && tile_width != esc::tma::Geom64::TW) return ESC_ERR_UNSUPPORTED;
    g_tile_policy = tile_width;
    return ESC_OK;
}
int esc_convattn_set_stencil_engine(int engine) {
    if (engine != ESC_ENGINE_AUTO && engine != ESC_ENGINE_FP32 && engine != ESC_ENGINE_TENSOR) return ESC_ERR_UNSUPPORTED;
    g_engine_policy = engine;
    return ESC_OK;
}
int esc_convattn_set_dense_engine(int engine) {
    if (engine != 0 && engine != 1) return ESC_ERR_UNSUPPORTED;
    g_dense_engine = engine;
    return ESC_OK;
}
int esc_convattn_set_fused_stage1(int on) {
    g_fuse_stage1 = on != 0;
    return ESC_OK;
}
int esc_convattn_last_launches(void) { return g_last_launches; }

const char* esc_status_string(int s) {
    switch (s) {
        case ESC_OK: return "ok";
        case ESC_ERR_NULL: return "null pointer";
        case ESC_ERR_SHAPE: return "invalid shape";
        case ESC_ERR_UNSUPPORTED: return "unsupported configuration";
        case ESC_ERR_ALIGN: return "misaligned pointer";
        case ESC_ERR_ALIAS: return "out overlaps x";
        case ESC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case ESC_ERR_CUDA: return "CUDA error";
        case ESC_DEV_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

size_t esc_convattn_workspace_bytes(int B, int C_a, int H, int W, int K) {
    if (B <= 0 || C_a <= 0 || H <= 0 || W <= 0 || K < 3 || (K & 1) == 0 || K > ESC_MAX_K) return 0;
    return workspace_bytes(B, C_a, (long long)H * W);
}

int esc_convattn_workspace_init(void* workspace, size_t workspace_bytes_, void* stream) {
    if (!workspace || !aligned(workspace, 256) || workspace_bytes_ < 256) return ESC_ERR_WORKSPACE;
    ESC_CUDA(cudaMemsetAsync(workspace, 0, workspace_bytes_, static_cast<cudaStream_t>(stream)));
    return ESC_OK;
}

int esc_convattn_forward_ex(const void* x, int B, int C, int C_a, int H, int W, int K, const void* w_large,
                            const void* w_dyn, const void* b_dyn, void* out, int dtype, int layout,
                            void* workspace, size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    const Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!w_large || !w_dyn || !b_dyn) return ESC_ERR_NULL;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_large, p.es()) || !aligned(w_dyn, p.es()) || !aligned(b_dyn, p.es())) return ESC_ERR_ALIGN;
    rc = check_workspace(p, workspace, workspace_bytes_);
    if (rc != ESC_OK) return rc;
    return forward_impl(p, x, w_large, Estimator{w_dyn, b_dyn, nullptr, nullptr, 0}, out, workspace,
                        static_cast<cudaStream_t>(stream));
}

int esc_convattn_forward(const void* x, int B, int C, int C_a, int H, int W, int K, const void* w_large,
                         const void* w_dyn, const void* b_dyn, void* out, void* stream) {
    g_last_launches = 0;
    const Problem p{B, C, C_a, H, W, K, ESC_F32, ESC_NCHW};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!w_large || !w_dyn || !b_dyn) return ESC_ERR_NULL;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_large, 4) || !aligned(w_dyn, 4) || !aligned(b_dyn, 4)) return ESC_ERR_ALIGN;
    void* ws = nullptr;
    rc = get_scratch(workspace_bytes(B, C_a, (long long)H * W), static_cast<cudaStream_t>(stream), &ws);
    if (rc != ESC_OK) return rc;
    return forward_impl(p, x, w_large, Estimator{w_dyn, b_dyn, nullptr, nullptr, 0}, out, ws, static_cast<cudaStream_t>(stream));
}

int esc_convattn_dynkernel(const void* x, int B, int C, int C_a, int H, int W, const void* w_dyn,
                           const void* b_dyn, float* dk_out, int dtype, int layout, void* workspace,
                           size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    const Problem p{B, C, C_a, H, W, 3, dtype, layout};   // stage 1 has no large kernel: any valid K
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!x || !w_dyn || !b_dyn || !dk_out) return ESC_ERR_NULL;
    if (!aligned(x, 16) || !aligned(dk_out, 4) || !aligned(w_dyn, p.es()) || !aligned(b_dyn, p.es())) return ESC_ERR_ALIGN;
    rc = check_workspace(p, workspace, workspace_bytes_);
    if (rc != ESC_OK) return rc;
    return launch_gap(p, x, Estimator{w_dyn, b_dyn, nullptr, nullptr, 0}, carve(workspace, B, C_a, (long long)H * W), dk_out,
                      static_cast<cudaStream_t>(stream));
}

int esc_convattn_forward_mlp(const void* x, int B, int C, int C_a, int H, int W, int K, const void* w_large,
                             const void* w_down, const void* b_down, const void* w_up, const void* b_up, int hidden,
                             void* out, int dtype, int layout, void* workspace, size_t workspace_bytes_,
                             void* stream) {
    g_last_launches = 0;
    const Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (hidden < 1) return ESC_ERR_SHAPE;
    if (!w_large) return ESC_ERR_NULL;
    const Estimator est{w_up, b_up, w_down, b_down, hidden};
    rc = check_estimator(p, est);
    if (rc != ESC_OK) return rc;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_large, p.es())) return ESC_ERR_ALIGN;
    rc = check_workspace(p, workspace, workspace_bytes_);
    if (rc != ESC_OK) return rc;
    return forward_impl(p, x, w_large, est, out, workspace, static_cast<cudaStream_t>(stream));
}

int esc_convattn_dynkernel_mlp(const void* x, int B, int C, int C_a, int H, int W, const void* w_down,
                               const void* b_down, const void* w_up, const void* b_up, int hidden, float* dk_out,
                               int dtype, int layout, void* workspace, size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    const Problem p{B, C, C_a, H, W, 3, dtype, layout};   // stage 1 has no large kernel: any valid K
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (hidden < 1) return ESC_ERR_SHAPE;
    if (!x || !dk_out) return ESC_ERR_NULL;
    const Estimator est{w_up, b_up, w_down, b_down, hidden};
    rc = check_estimator(p, est);
    if (rc != ESC_OK) return rc;
    if (!aligned(x, 16) || !aligned(dk_out, 4)) return ESC_ERR_ALIGN;
    rc = check_workspace(p, workspace, workspace_bytes_);
    if (rc != ESC_OK) return rc;
    return launch_gap(p, x, est, carve(workspace, B, C_a, (long long)H * W), dk_out, static_cast<cudaStream_t>(stream));
}

int esc_convattn_dynkernel_static(const void* x, int B, int C, int C_a, int H, int W, const void* w_dyn,
                                  const void* b_dyn, float* dk_out, int dtype, int layout, void* stream) {
    g_last_launches = 0;
    const Problem p{B, C, C_a, H, W, 3, dtype, layout};   // stage 1 has no large kernel: any valid K
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!x || !w_dyn || !b_dyn || !dk_out) return ESC_ERR_NULL;
    if (!aligned(x, 16) || !aligned(dk_out, 4) || !aligned(w_dyn, p.es()) || !aligned(b_dyn, p.es())) return ESC_ERR_ALIGN;
    const int S = slabs_for(B, (long long)H * W, wide_gap(B, (long long)H * W, false));
    if (B > kStaticMaxImages || (long long)B * S * C_a > kStaticMaxPartials) {
        char buf[200];
        snprintf(buf, sizeof buf,
                 "esc_convattn_dynkernel_static: needs %d counters and %lld partial sums, the fixed scratch holds %d and %d",
                 B, (long long)B * S * C_a, kStaticMaxImages, kStaticMaxPartials);
        g_last_error = buf;
        return ESC_ERR_WORKSPACE;
    }
    unsigned* base = nullptr;
    rc = static_scratch_address(&base);
    if (rc != ESC_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The counters must be zero when the kernel starts; a call that was cut short could have left them
    // otherwise, and the array is shared by every caller in the process.
    ESC_CUDA(cudaMemsetAsync(base, 0, (size_t)B * sizeof(unsigned), st));
    Workspace w;
    w.ctrl = nullptr;
    w.arrivals = base;
    w.dk = dk_out;
    w.partial = reinterpret_cast<float*>(base + kStaticMaxImages);
    return launch_gap(p, x, Estimator{w_dyn, b_dyn, nullptr, nullptr, 0}, w, dk_out, st);
}

int esc_convattn_stencil(const void* x, int B, int C, int C_a, int H, int W, int K, const void* w_large,
                         const float* dk, void* out, int dtype, int layout, void* workspace,
                         size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    const Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!w_large || !dk) return ESC_ERR_NULL;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_large, p.es()) || !aligned(dk, 4)) return ESC_ERR_ALIGN;
    unsigned* ctrl = nullptr;
    void* pad = nullptr;
    if (workspace) {
        rc = check_workspace(p, workspace, workspace_bytes_);
        if (rc != ESC_OK) return rc;
        const Workspace w = carve(workspace, B, C_a, (long long)H * W);
        ctrl = w.ctrl; pad = w.lk_pad;
    }
    const TensorLk tl = tensor_lk(p, x, out, w_large, pad, static_cast<cudaStream_t>(stream));
    return launch_stencil(p, x, w_large, dk, out, ctrl, static_cast<cudaStream_t>(stream), /*dependent=*/false, &tl);
}

int esc_convattn_stencil_pw(const void* x, int B, int C, int C_a, int H, int W, int K, const void* w_large,
                            const void* w_point, const float* dk, void* out, int dtype, int layout, void* workspace,
                            size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!w_large || !w_point || !dk) return ESC_ERR_NULL;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_large, p.es()) || !aligned(w_point, p.es()) || !aligned(dk, 4)) return ESC_ERR_ALIGN;
    p.w_point = w_point;
    unsigned* ctrl = nullptr;
    void* pad = nullptr;
    if (workspace) {
        rc = check_workspace(p, workspace, workspace_bytes_);
        if (rc != ESC_OK) return rc;
        const Workspace w = carve(workspace, B, C_a, (long long)H * W);
        ctrl = w.ctrl; pad = w.lk_pad;
    }
    const TensorLk tl = tensor_lk(p, x, out, w_large, pad, static_cast<cudaStream_t>(stream));
    return launch_stencil(p, x, w_large, dk, out, ctrl, static_cast<cudaStream_t>(stream), /*dependent=*/false, &tl);
}

int esc_convattn_forward_pw(const void* x, int B, int C, int C_a, int H, int W, int K, const void* w_large,
                            const void* w_point, const void* w_dyn, const void* b_dyn, void* out, int dtype,
                            int layout, void* workspace, size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!w_large || !w_point || !w_dyn || !b_dyn) return ESC_ERR_NULL;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_large, p.es()) || !aligned(w_point, p.es()) || !aligned(w_dyn, p.es()) || !aligned(b_dyn, p.es()))
        return ESC_ERR_ALIGN;
    rc = check_workspace(p, workspace, workspace_bytes_);
    if (rc != ESC_OK) return rc;
    p.w_point = w_point;
    return forward_impl(p, x, w_large, Estimator{w_dyn, b_dyn, nullptr, nullptr, 0}, out, workspace,
                        static_cast<cudaStream_t>(stream));
}

int esc_convattn_stencil_dense(const void* x, int B, int C, int C_a, int H, int W, int K, const void* w_dense,
                               const float* dk, void* out, int dtype, int layout, void* workspace,
                               size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!w_dense || !dk) return ESC_ERR_NULL;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_dense, p.es()) || !aligned(dk, 4)) return ESC_ERR_ALIGN;
    p.dense = true;
    unsigned* ctrl = nullptr;
    if (workspace) {
        rc = check_workspace(p, workspace, workspace_bytes_);
        if (rc != ESC_OK) return rc;
        ctrl = carve(workspace, B, C_a, (long long)H * W).ctrl;
    }
    return launch_stencil_dense(p, x, w_dense, dk, out, ctrl, static_cast<cudaStream_t>(stream), /*dependent=*/false);
}

int esc_convattn_forward_dense(const void* x, int B, int C, int C_a, int H, int W, int K, const void* w_dense,
                               const void* w_dyn, const void* b_dyn, void* out, int dtype, int layout,
                               void* workspace, size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!w_dense || !w_dyn || !b_dyn) return ESC_ERR_NULL;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_dense, p.es()) || !aligned(w_dyn, p.es()) || !aligned(b_dyn, p.es())) return ESC_ERR_ALIGN;
    rc = check_workspace(p, workspace, workspace_bytes_);
    if (rc != ESC_OK) return rc;
    p.dense = true;
    return forward_impl(p, x, w_dense, Estimator{w_dyn, b_dyn, nullptr, nullptr, 0}, out, workspace,
                        static_cast<cudaStream_t>(stream));
}

int esc_convattn_forward_variant(const void* x, int B, int C, int C_a, int H, int W, int K, int large_kernel,
                                 const void* w_large, const void* w_point, const void* w_down, const void* b_down,
                                 const void* w_up, const void* b_up, int hidden, void* out, int dtype, int layout,
                                 void* workspace, size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (large_kernel != ESC_LK_DEPTHWISE && large_kernel != ESC_LK_DECOMPOSED && large_kernel != ESC_LK_DENSE)
        return ESC_ERR_UNSUPPORTED;
    if (hidden < 0) return ESC_ERR_SHAPE;
    if (!w_large || (large_kernel == ESC_LK_DECOMPOSED && !w_point)) return ESC_ERR_NULL;
    const Estimator est{w_up, b_up, hidden > 0 ? w_down : nullptr, hidden > 0 ? b_down : nullptr, hidden};
    rc = check_estimator(p, est);
    if (rc != ESC_OK) return rc;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_large, p.es()) || (large_kernel == ESC_LK_DECOMPOSED && !aligned(w_point, p.es()))) return ESC_ERR_ALIGN;
    rc = check_workspace(p, workspace, workspace_bytes_);
    if (rc != ESC_OK) return rc;
    if (large_kernel == ESC_LK_DECOMPOSED) p.w_point = w_point;
    p.dense = large_kernel == ESC_LK_DENSE;
    return forward_impl(p, x, w_large, est, out, workspace, static_cast<cudaStream_t>(stream));
}

int esc_convattn_forward_fused(const void* x, int B, int C, int C_a, int H, int W, int K, const void* w_large,
                               const void* w_dyn, const void* b_dyn, const void* w_fuse, const void* b_fuse,
                               const void* residual, void* out, int dtype, int layout, void* workspace,
                               size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!w_large || !w_dyn || !b_dyn || !w_fuse) return ESC_ERR_NULL;
    rc = check_tensors(p, x, out);
    if (rc != ESC_OK) return rc;
    if (!aligned(w_large, p.es()) || !aligned(w_dyn, p.es()) || !aligned(b_dyn, p.es()) || !aligned(w_fuse, p.es()) ||
        (b_fuse && !aligned(b_fuse, p.es())))
        return ESC_ERR_ALIGN;
    if (residual) {
        if (!aligned(residual, 16)) return ESC_ERR_ALIGN;
        const uintptr_t ra = reinterpret_cast<uintptr_t>(residual), oa = reinterpret_cast<uintptr_t>(out);
        const size_t bytes = p.elems() * p.es();
        if (ra < oa + bytes && oa < ra + bytes) return ESC_ERR_ALIAS;        // out is rewritten pixel block by pixel block
    }
    rc = check_workspace(p, workspace, workspace_bytes_);
    if (rc != ESC_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Estimator est{w_dyn, b_dyn, nullptr, nullptr, 0};
    const long long pixels = (long long)B * H * W;
    // Fast path: the tensor-core stencil writes only the attention channels; the 1x1 kernel takes the identity
    // channels straight from x, so they are never copied.
    if (esc::fuse::fast_applies(C, C_a, dtype, layout) && aligned(w_fuse, 16) && tensor_stencil_follows(p)) {
        p.skip_copy = true;
        rc = forward_impl(p, x, w_large, est, out, workspace, st);
        if (rc != ESC_OK) return rc;
        esc::fuse::Params fp;
        fp.att = static_cast<const __nv_bfloat16*>(out); fp.idt = static_cast<const __nv_bfloat16*>(x);
        fp.w = static_cast<const __nv_bfloat16*>(w_fuse); fp.bias = static_cast<const __nv_bfloat16*>(b_fuse);
        fp.residual = static_cast<const __nv_bfloat16*>(residual); fp.out = static_cast<__nv_bfloat16*>(out);
        fp.pixels = pixels; fp.C = C; fp.Ca = C_a;
        ESC_CUDA(esc::fuse::launch_fast(fp, st));
        ++g_last_launches;
        return ESC_OK;
    }
    // The same on NCHW tensors: the NCHW tensor-core stencil without its copy of the identity planes, then the NCHW 1x1 kernel.
    if (K == esc::tma::K13 && g_engine_policy != ESC_ENGINE_FP32 && g_tile_policy == 0 &&
        esc::fuse::nchw::applies(C, C_a, (long long)H * W, dtype, layout, x, out, residual, w_fuse) &&
        esc::tma::toepn::applies(C, C_a, H, W, K, dtype, layout, x, out)) {
        p.skip_copy = true;
        rc = forward_impl(p, x, w_large, est, out, workspace, st);
        if (rc != ESC_OK) return rc;
        esc::fuse::nchw::Params fp;
        fp.att = static_cast<const __nv_bfloat16*>(out); fp.idt = static_cast<const __nv_bfloat16*>(x);
        fp.w = static_cast<const __nv_bfloat16*>(w_fuse); fp.bias = static_cast<const __nv_bfloat16*>(b_fuse);
        fp.residual = static_cast<const __nv_bfloat16*>(residual); fp.out = static_cast<__nv_bfloat16*>(out);
        fp.HW = (long long)H * W; fp.B = B; fp.C = C; fp.Ca = C_a;
        ESC_CUDA(esc::fuse::nchw::launch(fp, st));
        ++g_last_launches;
        return ESC_OK;
    }
    rc = forward_impl(p, x, w_large, est, out, workspace, st);
    if (rc != ESC_OK) return rc;
    const size_t smem = (size_t)esc::fuse::kGenPix * C * sizeof(float);
    if (smem > 48 * 1024) return ESC_ERR_UNSUPPORTED;
    const unsigned blocks = (unsigned)((pixels + esc::fuse::kGenPix - 1) / esc::fuse::kGenPix);
#define ESC_FUSE_GENERIC(T, L) esc::fuse::conv_fuse_generic<T, L><<<blocks, esc::fuse::kGenThreads, smem, st>>>( \
        static_cast<T*>(out), static_cast<const T*>(w_fuse), static_cast<const T*>(b_fuse), static_cast<const T*>(residual), B, C, H, W)
    if (dtype == ESC_F32) { if (layout == ESC_NCHW) ESC_FUSE_GENERIC(float, esc::kNCHW); else ESC_FUSE_GENERIC(float, esc::kNHWC); }
    else { if (layout == ESC_NCHW) ESC_FUSE_GENERIC(__nv_bfloat16, esc::kNCHW); else ESC_FUSE_GENERIC(__nv_bfloat16, esc::kNHWC); }
#undef ESC_FUSE_GENERIC
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    return ESC_OK;
}

size_t esc_convattn_backward_workspace_bytes(int B, int C_a, int H, int W, int K) {
    if (B <= 0 || C_a <= 0 || H <= 0 || W <= 0 || K < 3 || K > esc::bwd::K || (K & 1) == 0) return 0;
    const Problem p{B, C_a, C_a, H, W, K, ESC_F32, ESC_NCHW};
    return carve_backward(nullptr, p).bytes;
}

namespace {
int backward_entry(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K, const void* w_large,
                   const Estimator& est, void* grad_x, const BackwardGrads& g, int dtype, int layout, void* workspace,
                   size_t workspace_bytes_, void* stream, const void* w_point = nullptr, float* g_wp = nullptr,
                   bool dense = false, float* g_wd = nullptr) {
    g_last_launches = 0;
    Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (K > esc::bwd::K) return ESC_ERR_UNSUPPORTED;         // the tap-gradient kernels hold 13 x 13 taps; a smaller LK is their middle
    if ((long long)B * C_a > 0x7fffffffLL / esc::bwd::kSlot) return ESC_ERR_UNSUPPORTED;
    if (!x || !grad_out || !grad_x || !w_large) return ESC_ERR_NULL;
    rc = check_estimator(p, est);
    if (rc != ESC_OK) return rc;
    rc = check_tensors(p, grad_out, grad_x);                 // the stencil pass reads grad_out and writes grad_x
    if (rc != ESC_OK) return rc;
    if (!aligned(x, 16)) return ESC_ERR_ALIGN;
    {
        const uintptr_t xa = reinterpret_cast<uintptr_t>(x), oa = reinterpret_cast<uintptr_t>(grad_x);
        const size_t bytes = p.elems() * p.es();
        if (xa < oa + bytes && oa < xa + bytes) return ESC_ERR_ALIAS;
    }
    if (!aligned(w_large, p.es())) return ESC_ERR_ALIGN;
    for (const float* q : {g.g_lk, g.g_w_last, g.g_b_last, g.g_w_down, g.g_b_down, g_wp})
        if (q && !aligned(q, 4)) return ESC_ERR_ALIGN;
    if (w_point) {
        if (!aligned(w_point, p.es())) return ESC_ERR_ALIGN;
        if (!esc::bwd::pw::supported(C_a)) return ESC_ERR_UNSUPPORTED;
        if ((long long)B * esc::bwd::pw::chunks_of((long long)H * W) > 0x7fffffffLL) return ESC_ERR_UNSUPPORTED;
    }
    if (!workspace || !aligned(workspace, 256)) return ESC_ERR_WORKSPACE;
    if (dense && (C_a != esc::bwd::dense::CA || w_point)) return ESC_ERR_UNSUPPORTED;
    if (g_wd && !aligned(g_wd, 4)) return ESC_ERR_ALIGN;
    BackwardWs w = carve_backward(workspace, p);
    if (workspace_bytes_ < (dense ? w.bytes_dense : w.bytes)) return ESC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (w_point) {
        // decomposed form (Eq. 5): the mixed features go into grad_x's attention channels, where the tap-gradient kernels
        // read them; grad_x is rewritten by the stencil pass and the last kernel below
        rc = dtype == ESC_F32 ? (layout == ESC_NCHW ? pw_mix_t<float, esc::kNCHW>(p, x, w_point, grad_x, w, st)
                                                    : pw_mix_t<float, esc::kNHWC>(p, x, w_point, grad_x, w, st))
                              : (layout == ESC_NCHW ? pw_mix_t<__nv_bfloat16, esc::kNCHW>(p, x, w_point, grad_x, w, st)
                                                    : pw_mix_t<__nv_bfloat16, esc::kNHWC>(p, x, w_point, grad_x, w, st));
        if (rc != ESC_OK) return rc;
        w.patch_xsum = true;
    }
    const void* x_taps = w_point ? grad_x : x;             // what the depth-wise stage saw
    if (dense) {
        // w_large is the dense kernel [16][16][K][K]: its gradient and its rotated form here; the depth-wise kernels
        // below give g_dk (the middle 3 x 3 of their tap gradients) and what follows from it
        rc = dtype == ESC_F32 ? (layout == ESC_NCHW ? dense_tap_grad_t<float, esc::kNCHW>(p, x, grad_out, w_large, w, g_wd, st)
                                                    : dense_tap_grad_t<float, esc::kNHWC>(p, x, grad_out, w_large, w, g_wd, st))
                              : (layout == ESC_NCHW ? dense_tap_grad_t<__nv_bfloat16, esc::kNCHW>(p, x, grad_out, w_large, w, g_wd, st)
                                                    : dense_tap_grad_t<__nv_bfloat16, esc::kNHWC>(p, x, grad_out, w_large, w, g_wd, st));
        if (rc != ESC_OK) return rc;
    }
    if (dtype == ESC_F32)
        rc = layout == ESC_NCHW ? backward_t<float, esc::kNCHW>(p, x_taps, grad_out, w_large, est, w, g, st)
                                : backward_t<float, esc::kNHWC>(p, x_taps, grad_out, w_large, est, w, g, st);
    else
        rc = layout == ESC_NCHW ? backward_t<__nv_bfloat16, esc::kNCHW>(p, x_taps, grad_out, w_large, est, w, g, st)
                                : backward_t<__nv_bfloat16, esc::kNHWC>(p, x_taps, grad_out, w_large, est, w, g, st);
    if (rc != ESC_OK) return rc;
    // grad_x: the forward stencil on grad_out with both kernels rotated by 180 degrees, plus the constants (in the
    // decomposed form the constants belong behind the transposed mix: the last kernel adds them)
    if (dense) {
        p.dense = true;
        rc = launch_stencil_dense(p, grad_out, w.wd_flip, w.dk_flip, grad_x, w.ctrl, st, /*dependent=*/false);
        if (rc != ESC_OK) return rc;
        return dtype == ESC_F32 ? (layout == ESC_NCHW ? dense_add_const_t<float, esc::kNCHW>(p, grad_x, w, st)
                                                      : dense_add_const_t<float, esc::kNHWC>(p, grad_x, w, st))
                                : (layout == ESC_NCHW ? dense_add_const_t<__nv_bfloat16, esc::kNCHW>(p, grad_x, w, st)
                                                      : dense_add_const_t<__nv_bfloat16, esc::kNHWC>(p, grad_x, w, st));
    }
    p.bias = w_point ? nullptr : w.bias;
    const TensorLk tl = tensor_lk(p, grad_out, grad_x, w.w_flip, w.lk_pad, st);
    rc = launch_stencil(p, grad_out, w.w_flip, w.dk_flip, grad_x, w.ctrl, st, /*dependent=*/false, &tl);
    if (rc != ESC_OK || !w_point) return rc;
    rc = dtype == ESC_F32 ? (layout == ESC_NCHW ? pw_back_t<float, esc::kNCHW>(p, x, w_point, grad_x, w, g_wp, st)
                                                : pw_back_t<float, esc::kNHWC>(p, x, w_point, grad_x, w, g_wp, st))
                          : (layout == ESC_NCHW ? pw_back_t<__nv_bfloat16, esc::kNCHW>(p, x, w_point, grad_x, w, g_wp, st)
                                                : pw_back_t<__nv_bfloat16, esc::kNHWC>(p, x, w_point, grad_x, w, g_wp, st));
    return rc;
}
}  // namespace

int esc_convattn_backward(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                          const void* w_large, const void* w_dyn, const void* b_dyn, void* grad_x,
                          float* grad_w_large, float* grad_w_dyn, float* grad_b_dyn, int dtype, int layout,
                          void* workspace, size_t workspace_bytes_, void* stream) {
    const Estimator est{w_dyn, b_dyn, nullptr, nullptr, 0};
    const BackwardGrads g{grad_w_large, grad_w_dyn, grad_b_dyn, nullptr, nullptr};
    return backward_entry(x, grad_out, B, C, C_a, H, W, K, w_large, est, grad_x, g, dtype, layout, workspace, workspace_bytes_, stream);
}

int esc_convattn_backward_mlp(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                              const void* w_large, const void* w_down, const void* b_down, const void* w_up,
                              const void* b_up, int hidden, void* grad_x, float* grad_w_large, float* grad_w_down,
                              float* grad_b_down, float* grad_w_up, float* grad_b_up, int dtype, int layout,
                              void* workspace, size_t workspace_bytes_, void* stream) {
    if (hidden <= 0) return ESC_ERR_SHAPE;
    const Estimator est{w_up, b_up, w_down, b_down, hidden};
    const BackwardGrads g{grad_w_large, grad_w_up, grad_b_up, grad_w_down, grad_b_down};
    return backward_entry(x, grad_out, B, C, C_a, H, W, K, w_large, est, grad_x, g, dtype, layout, workspace, workspace_bytes_, stream);
}

int esc_convattn_backward_pw(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                             const void* w_large, const void* w_point, const void* w_dyn, const void* b_dyn, void* grad_x,
                             float* grad_w_large, float* grad_w_point, float* grad_w_dyn, float* grad_b_dyn, int dtype,
                             int layout, void* workspace, size_t workspace_bytes_, void* stream) {
    if (!w_point) return ESC_ERR_NULL;
    const Estimator est{w_dyn, b_dyn, nullptr, nullptr, 0};
    const BackwardGrads g{grad_w_large, grad_w_dyn, grad_b_dyn, nullptr, nullptr};
    return backward_entry(x, grad_out, B, C, C_a, H, W, K, w_large, est, grad_x, g, dtype, layout, workspace, workspace_bytes_, stream,
                          w_point, grad_w_point);
}

size_t esc_convattn_backward_dense_workspace_bytes(int B, int C_a, int H, int W, int K) {
    if (B <= 0 || C_a != esc::bwd::dense::CA || H <= 0 || W <= 0 || K < 3 || K > esc::bwd::K || (K & 1) == 0) return 0;
    const Problem p{B, C_a, C_a, H, W, K, ESC_F32, ESC_NCHW};
    return carve_backward(nullptr, p).bytes_dense;
}

int esc_convattn_backward_dense(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                                const void* w_dense, const void* w_dyn, const void* b_dyn, void* grad_x,
                                float* grad_w_dense, float* grad_w_dyn, float* grad_b_dyn, int dtype, int layout,
                                void* workspace, size_t workspace_bytes_, void* stream) {
    const Estimator est{w_dyn, b_dyn, nullptr, nullptr, 0};
    const BackwardGrads g{nullptr, grad_w_dyn, grad_b_dyn, nullptr, nullptr};
    return backward_entry(x, grad_out, B, C, C_a, H, W, K, w_dense, est, grad_x, g, dtype, layout, workspace, workspace_bytes_, stream,
                          nullptr, nullptr, /*dense=*/true, grad_w_dense);
}

int esc_convattn_backward_variant(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                                  int large_kernel, const void* w_large, const void* w_point, const void* w_down,
                                  const void* b_down, const void* w_up, const void* b_up, int hidden, void* grad_x,
                                  float* grad_w_large, float* grad_w_point, float* grad_w_down, float* grad_b_down,
                                  float* grad_w_up, float* grad_b_up, int dtype, int layout, void* workspace,
                                  size_t workspace_bytes_, void* stream) {
    if (large_kernel != ESC_LK_DEPTHWISE && large_kernel != ESC_LK_DECOMPOSED && large_kernel != ESC_LK_DENSE)
        return ESC_ERR_UNSUPPORTED;
    if (hidden < 0) return ESC_ERR_SHAPE;
    if (large_kernel == ESC_LK_DECOMPOSED && !w_point) return ESC_ERR_NULL;
    const Estimator est{w_up, b_up, hidden > 0 ? w_down : nullptr, hidden > 0 ? b_down : nullptr, hidden};
    const bool dense = large_kernel == ESC_LK_DENSE;
    const BackwardGrads g{dense ? nullptr : grad_w_large, grad_w_up, grad_b_up, hidden > 0 ? grad_w_down : nullptr,
                          hidden > 0 ? grad_b_down : nullptr};
    return backward_entry(x, grad_out, B, C, C_a, H, W, K, w_large, est, grad_x, g, dtype, layout, workspace, workspace_bytes_, stream,
                          large_kernel == ESC_LK_DECOMPOSED ? w_point : nullptr,
                          large_kernel == ESC_LK_DECOMPOSED ? grad_w_point : nullptr, dense, dense ? grad_w_large : nullptr);
}

size_t esc_conv_fuse_backward_workspace_bytes(int B, int C, int H, int W) {
    if (B <= 0 || H <= 0 || W <= 0 || !esc::fuse::bwd::supported(C)) return 0;
    return carve_fuse_backward(nullptr, C, (long long)B * H * W).bytes;
}

int esc_conv_fuse_backward(const void* cat, const void* grad_out, int B, int C, int H, int W, const void* w_fuse,
                           void* grad_cat, float* grad_w_fuse, float* grad_b_fuse, int dtype, int layout,
                           void* workspace, size_t workspace_bytes_, void* stream) {
    g_last_launches = 0;
    const Problem p{B, C, C, H, W, 3, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!esc::fuse::bwd::supported(C)) return ESC_ERR_UNSUPPORTED;
    if (!cat || !grad_out || !w_fuse || !grad_cat) return ESC_ERR_NULL;
    rc = check_tensors(p, grad_out, grad_cat);
    if (rc != ESC_OK) return rc;
    if (!aligned(cat, 16) || !aligned(w_fuse, p.es())) return ESC_ERR_ALIGN;
    {
        const uintptr_t xa = reinterpret_cast<uintptr_t>(cat), oa = reinterpret_cast<uintptr_t>(grad_cat);
        const size_t bytes = p.elems() * p.es();
        if (xa < oa + bytes && oa < xa + bytes) return ESC_ERR_ALIAS;
    }
    for (const float* q : {grad_w_fuse, grad_b_fuse})
        if (q && !aligned(q, 4)) return ESC_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256)) return ESC_ERR_WORKSPACE;
    const long long HW = (long long)H * W, pixels = (long long)B * HW;
    const FuseBackwardWs w = carve_fuse_backward(workspace, C, pixels);
    if (workspace_bytes_ < w.bytes) return ESC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the weight's and the bias's gradients
    if (grad_w_fuse || grad_b_fuse) {
        if (dtype == ESC_F32)
            rc = layout == ESC_NCHW ? fuse_wgrad_t<float, esc::kNCHW>(C, cat, grad_out, HW, pixels, w, st)
                                    : fuse_wgrad_t<float, esc::kNHWC>(C, cat, grad_out, HW, pixels, w, st);
        else
            rc = layout == ESC_NCHW ? fuse_wgrad_t<__nv_bfloat16, esc::kNCHW>(C, cat, grad_out, HW, pixels, w, st)
                                    : fuse_wgrad_t<__nv_bfloat16, esc::kNHWC>(C, cat, grad_out, HW, pixels, w, st);
        if (rc != ESC_OK) return rc;
        const int elems = C * C + C;
        esc::fuse::bwd::sum_wgrad<<<(unsigned)((elems + 7) / 8), 256, 0, st>>>(w.part, C, w.blocks, grad_w_fuse, grad_b_fuse);
        ESC_CUDA(cudaGetLastError());
        ++g_last_launches;
    }
    // grad_cat = W_fuse^T grad_out per pixel: the forward's 1x1 kernels with the transposed matrix, no bias, no residual
    const unsigned tb = (unsigned)((C * C + 255) / 256);
    if (dtype == ESC_F32) esc::fuse::bwd::transpose_w<float><<<tb, 256, 0, st>>>(static_cast<const float*>(w_fuse), C, static_cast<float*>(w.wt));
    else esc::fuse::bwd::transpose_w<__nv_bfloat16><<<tb, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(w_fuse), C, static_cast<__nv_bfloat16*>(w.wt));
    ESC_CUDA(cudaGetLastError());
    ++g_last_launches;
    if (esc::fuse::fast_applies(C, 8, dtype, layout)) {
        esc::fuse::Params fp;
        fp.att = static_cast<const __nv_bfloat16*>(grad_out); fp.idt = static_cast<const __nv_bfloat16*>(grad_out);
        fp.w = static_cast<const __nv_bfloat16*>(w.wt); fp.bias = nullptr; fp.residual = nullptr;
        fp.out = static_cast<__nv_bfloat16*>(grad_cat);
        fp.pixels = pixels; fp.C = C; fp.Ca = 8;
        ESC_CUDA(esc::fuse::launch_fast(fp, st, /*early=*/false));   // its matrix was written by the kernel before it
        ++g_last_launches;
        return ESC_OK;
    }
    if (esc::fuse::nchw::applies(C, 8, HW, dtype, layout, grad_out, grad_cat, nullptr, w.wt)) {
        esc::fuse::nchw::Params fp;
        fp.att = static_cast<const __nv_bfloat16*>(grad_out); fp.idt = static_cast<const __nv_bfloat16*>(grad_out);
        fp.w = static_cast<const __nv_bfloat16*>(w.wt); fp.bias = nullptr; fp.residual = nullptr;
        fp.out = static_cast<__nv_bfloat16*>(grad_cat);
        fp.HW = HW; fp.B = B; fp.C = C; fp.Ca = 8;
        ESC_CUDA(esc::fuse::nchw::launch(fp, st, /*early=*/false));
        ++g_last_launches;
        return ESC_OK;
    }
    // any type and layout: the generic kernel works in place on a copy of grad_out
    ESC_CUDA(cudaMemcpyAsync(grad_cat, grad_out, p.elems() * p.es(), cudaMemcpyDeviceToDevice, st));
    const size_t smem = (size_t)esc::fuse::kGenPix * C * sizeof(float);
    const unsigned blocks = (unsigned)((pixels + esc::fuse::kGenPix - 1) / esc::fuse::kGenPix);
#define ESC_FUSE_GENERIC(T, L) esc::fuse::conv_fuse_generic<T, L><<<blocks, esc::fuse::kGenThreads, smem, st>>>( \
        static_cast<T*>(grad_cat), static_cast<const T*>(w.wt), static_cast<const T*>(nullptr), static_cast<const T*>(nullptr), B, C, H, W)
    if (dtype == ESC_F32) { if (layout == ESC_NCHW) ESC_FUSE_GENERIC(float, esc::kNCHW); else ESC_FUSE_GENERIC(float, esc::kNHWC); }
    else { if (layout == ESC_NCHW) ESC_FUSE_GENERIC(__nv_bfloat16, esc::kNCHW); else ESC_FUSE_GENERIC(__nv_bfloat16, esc::kNHWC); }
#undef ESC_FUSE_GENERIC
    ESC_CUDA(cudaGetLastError());
    g_last_launches += 2;
    return ESC_OK;
}

int esc_convattn_selftest_bounded_wait(void* workspace, void* stream) {
    if (!workspace || !aligned(workspace, 256)) return ESC_ERR_WORKSPACE;
    bounded_wait_probe<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<unsigned*>(workspace));
    ESC_CUDA(cudaGetLastError());
    return ESC_OK;
}

int esc_convattn_device_status(void* workspace, void* stream) {
    if (!workspace) return ESC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned word[2] = {0, 0};
    ESC_CUDA(cudaMemcpyAsync(word, workspace, sizeof word, cudaMemcpyDeviceToHost, st));
    ESC_CUDA(cudaStreamSynchronize(st));
    if (word[0] != 0) {
        char buf[96];
        snprintf(buf, sizeof buf, "device status %u, detail 0x%x", word[0], word[1]);
        g_last_error = buf;
        ESC_CUDA(cudaMemsetAsync(workspace, 0, sizeof word, st));
        ESC_CUDA(cudaStreamSynchronize(st));
    }
    return (int)word[0];
}

int esc_convattn_forward_host_submit(int slot, const void* x_host, int B, int C, int C_a, int H, int W, int K,
                                     const void* w_large_host, const void* w_dyn_host, const void* b_dyn_host,
                                     void* out_host, int dtype, int layout) {
    g_last_launches = 0;
    if (slot < 0 || slot >= kHostSlots) return ESC_ERR_UNSUPPORTED;
    const Problem p{B, C, C_a, H, W, K, dtype, layout};
    int rc = check_shape(p);
    if (rc != ESC_OK) return rc;
    if (!x_host || !w_large_host || !w_dyn_host || !b_dyn_host || !out_host) return ESC_ERR_NULL;
    std::lock_guard<std::mutex> lock(g_host_mu);
    HostPath& h = g_host[slot];
    int dev = 0;
    ESC_CUDA(cudaGetDevice(&dev));
    if (h.dev != dev) {   // first use, or the caller switched device: start over
        if (h.dev >= 0) {
            ESC_CUDA(cudaSetDevice(h.dev));
            if (h.st) cudaStreamSynchronize(h.st);
            cudaFree(h.x); cudaFree(h.out); cudaFree(h.wts); cudaFree(h.ws);
            if (h.st) cudaStreamDestroy(h.st);
            ESC_CUDA(cudaSetDevice(dev));
        }
        h = HostPath();
        h.dev = dev;
        ESC_CUDA(cudaStreamCreateWithFlags(&h.st, cudaStreamNonBlocking));
    }
    const size_t es = p.es(), xbytes = p.elems() * es;
    const size_t n_wl = (size_t)C_a * K * K, n_wd = (size_t)9 * C_a * C_a, n_bd = (size_t)9 * C_a;
    const size_t off_wd = round_up(n_wl * es, 256), off_bd = off_wd + round_up(n_wd * es, 256);
    const size_t wbytes = off_bd + round_up(n_bd * es, 256);
    const size_t wsbytes = workspace_bytes(B, C_a, (long long)H * W);
    if (h.xbytes < xbytes || h.wbytes < wbytes || h.wsbytes < wsbytes)
        ESC_CUDA(cudaStreamSynchronize(h.st));               // nothing of this slot may still use the old buffers
    if (h.xbytes < xbytes) {
        cudaFree(h.x); cudaFree(h.out); h.x = h.out = nullptr; h.xbytes = 0;
        ESC_CUDA(cudaMalloc(&h.x, xbytes));
        ESC_CUDA(cudaMalloc(&h.out, xbytes));
        h.xbytes = xbytes;
    }
    if (h.wbytes < wbytes) {
        cudaFree(h.wts); h.wts = nullptr; h.wbytes = 0;
        ESC_CUDA(cudaMalloc(&h.wts, wbytes));
        h.wbytes = wbytes;
    }
    if (h.wsbytes < wsbytes) {
        cudaFree(h.ws); h.ws = nullptr; h.wsbytes = 0;
        ESC_CUDA(cudaMalloc(&h.ws, wsbytes));
        ESC_CUDA(cudaMemset(h.ws, 0, wsbytes));
        h.wsbytes = wsbytes;
    }
    char* wts = static_cast<char*>(h.wts);
    ESC_CUDA(cudaMemcpyAsync(h.x, x_host, xbytes, cudaMemcpyHostToDevice, h.st));
    ESC_CUDA(cudaMemcpyAsync(wts, w_large_host, n_wl * es, cudaMemcpyHostToDevice, h.st));
    ESC_CUDA(cudaMemcpyAsync(wts + off_wd, w_dyn_host, n_wd * es, cudaMemcpyHostToDevice, h.st));
    ESC_CUDA(cudaMemcpyAsync(wts + off_bd, b_dyn_host, n_bd * es, cudaMemcpyHostToDevice, h.st));
    rc = forward_impl(p, h.x, wts, Estimator{wts + off_wd, wts + off_bd, nullptr, nullptr, 0}, h.out, h.ws, h.st);
    if (rc != ESC_OK) return rc;
    ESC_CUDA(cudaMemcpyAsync(out_host, h.out, xbytes, cudaMemcpyDeviceToHost, h.st));
    return ESC_OK;
}

int esc_convattn_forward_host_wait(int slot) {
    if (slot < 0 || slot >= kHostSlots) return ESC_ERR_UNSUPPORTED;
    cudaStream_t st = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_host_mu);
        if (g_host[slot].dev < 0) return ESC_OK;             // nothing was ever submitted here
        st = g_host[slot].st;
    }
    ESC_CUDA(cudaStreamSynchronize(st));
    return ESC_OK;
}

int esc_convattn_forward_host(const void* x_host, int B, int C, int C_a, int H, int W, int K,
                              const void* w_large_host, const void* w_dyn_host, const void* b_dyn_host,
                              void* out_host, int dtype, int layout) {
    int rc = esc_convattn_forward_host_submit(0, x_host, B, C, C_a, H, W, K, w_large_host, w_dyn_host, b_dyn_host,
                                              out_host, dtype, layout);
    if (rc != ESC_OK) return rc;
    return esc_convattn_forward_host_wait(0);
}

}  // extern "C"

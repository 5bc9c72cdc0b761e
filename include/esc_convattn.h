/*
 * esc_convattn.h -- C ABI of the B200 (sm_100a) ConvAttn forward library.
 *
 * The operation is the Convolutional Attention module of the ESC paper
 * (Section 3.3, Eq. 4), in the depth-wise large-kernel form of Eq. 5 (LK^s, without the
 * point-wise LK^c) and with the kernel estimator reduced to one linear layer:
 *
 *   F_att = x[:, :C_a],  F_idt = x[:, C_a:]                               (Eq. 4, line 1)
 *   g[b,c]  = mean_{y,x} F_att[b,c,y,x]                                   (GAP, Eq. 4 line 2)
 *   dk[b,o] = b_dyn[o] + sum_c w_dyn[o,c] * g[b,c],   o = c*9 + i*3 + j   (Eq. 4 line 2)
 *   out[b,c,y,x] = sum_{i,j<K} w_large[c,i,j] * xp[b,c,y+i-P,x+j-P]
 *                + sum_{i,j<3} dk[b,c,i,j]    * xp[b,c,y+i-1,x+j-1]       (Eq. 4 line 3)
 *   out[b, C_a:] = F_idt, bit for bit                                     (Concat, Eq. 4 line 4)
 *
 * with P = (K-1)/2, xp = x extended by zeros ('same' padding) and the sums taken as
 * cross-correlations (no kernel flip).  Internally the two kernels are merged as
 * ZP(dk) + LK^s (Eq. 5).  g, dk and every accumulation are fp32; each output is rounded
 * once (round-to-nearest-even) to the storage type.
 *
 * General rules
 *  - Every function returns an esc_status (0 = success).  Nothing throws or aborts.
 *  - All tensor pointers are DEVICE pointers unless a parameter is named *_host.
 *    The caller owns every buffer; the library keeps no reference after the work that a
 *    call enqueued has finished.
 *  - Logical tensor shape is always [B,C,H,W]; `layout` says how it sits in memory
 *    (ESC_NCHW: dense [B][C][H][W];  ESC_NHWC: dense [B][H][W][C], PyTorch channels_last).
 *    Strides are dense.  Weights have the same element type as x.
 *  - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the legacy
 *    default stream).  Errors found on the host are returned at once and nothing is
 *    enqueued.  Device-side conditions (a bounded wait that expired) are recorded in the
 *    workspace status word and read back with esc_convattn_device_status().
 *  - Two calls may overlap on the GPU only if they use different workspaces.
 */
#ifndef ESC_CONVATTN_H
#define ESC_CONVATTN_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ESC_OK = 0,
    ESC_ERR_NULL = 1,        /* a required pointer is NULL                                      */
    ESC_ERR_SHAPE = 2,       /* B,C,H,W <= 0, C_a <= 0, C_a > C, K even or K < 3, size overflow */
    ESC_ERR_UNSUPPORTED = 3, /* K > ESC_MAX_K, unknown dtype / layout                           */
    ESC_ERR_ALIGN = 4,       /* a tensor pointer is not aligned to its element size / 16 bytes  */
    ESC_ERR_ALIAS = 5,       /* out overlaps x (a stencil cannot run in place)                  */
    ESC_ERR_WORKSPACE = 6,   /* workspace NULL, misaligned or smaller than required             */
    ESC_ERR_CUDA = 7,        /* a CUDA runtime / driver call failed; text in esc_last_error()   */
    ESC_DEV_TIMEOUT = 8      /* a bounded device-side wait expired (status word)                */
} esc_status;

enum { ESC_F32 = 0, ESC_BF16 = 1 };   /* element type of x, out and the three weight tensors */
enum { ESC_NCHW = 0, ESC_NHWC = 1 };  /* memory layout of x and out                           */
enum { ESC_MAX_K = 17 };              /* largest supported large-kernel size (odd)            */

/*
 * ConvAttn forward, Eq. 4 of the paper as restated above.  fp32 tensors in dense NCHW.
 *   x        [B,C,H,W]   input feature map (device, 16-byte aligned)
 *   w_large  [C_a,K,K]   shared depth-wise large kernel LK^s (K odd, <= ESC_MAX_K)
 *   w_dyn    [9*C_a,C_a] kernel-estimator weight, row o = c*9 + i*3 + j
 *   b_dyn    [9*C_a]     kernel-estimator bias
 *   out      [B,C,H,W]   result (device, 16-byte aligned, must not overlap x)
 * Scratch memory is owned by the library (one block per device and stream, created on
 * first use with cudaMalloc and kept until the process exits).
 */
int esc_convattn_forward(const void* x, int B, int C, int C_a, int H, int W, int K,
                         const void* w_large, const void* w_dyn, const void* b_dyn,
                         void* out, void* stream);

/*
 * Same operation with explicit element type, layout and caller-owned scratch.
 *   dtype      ESC_F32 or ESC_BF16 (bf16 storage, fp32 arithmetic)
 *   layout     ESC_NCHW or ESC_NHWC
 *   workspace  device memory of at least esc_convattn_workspace_bytes(...) bytes, 256-byte
 *              aligned, prepared once with esc_convattn_workspace_init(); it may be reused by
 *              later calls that do not overlap this one on the GPU.
 */
int esc_convattn_forward_ex(const void* x, int B, int C, int C_a, int H, int W, int K,
                            const void* w_large, const void* w_dyn, const void* b_dyn,
                            void* out, int dtype, int layout,
                            void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of scratch needed by the calls that take a workspace (dk, GAP partial sums,
 * arrival counters, status word).  Returns 0 for invalid arguments. */
size_t esc_convattn_workspace_bytes(int B, int C_a, int H, int W, int K);

/* Zero a fresh workspace (enqueued on `stream`).  Needed once per allocation; the kernels
 * leave the control words ready for the next call. */
int esc_convattn_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * Stage 1 alone (GAP + kernel estimator, Eq. 4 line 2): writes dk_out [B,C_a,3,3] fp32.
 */
int esc_convattn_dynkernel(const void* x, int B, int C, int C_a, int H, int W,
                           const void* w_dyn, const void* b_dyn, float* dk_out,
                           int dtype, int layout,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * The forward pass with the kernel estimator exactly as Eq. 4 line 2 of the paper writes it:
 *   DK = Conv_up(phi(Conv_down(GAP(F_att)))),  phi(t) = t * Phi(t)  (Gaussian error linear unit,
 * exact form through erfc, not the tanh approximation); both 1x1 convolutions carry a bias
 * (pass zeros for a bias-free estimator).  Section 3.3 sets the hidden width h to 4 or 8, the
 * larger model of the appendix to 24.
 *   w_down  [hidden,C_a]    b_down [hidden]
 *   w_up    [9*C_a,hidden]  b_up   [9*C_a]      row o = c*9 + i*3 + j, 1 <= hidden <= 128
 * All four in the tensor's dtype on the device; everything else as for esc_convattn_forward_ex,
 * including the workspace size.  ESC_ERR_SHAPE for hidden outside 1..128.
 */
int esc_convattn_forward_mlp(const void* x, int B, int C, int C_a, int H, int W, int K,
                             const void* w_large, const void* w_down, const void* b_down,
                             const void* w_up, const void* b_up, int hidden,
                             void* out, int dtype, int layout,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Stage 1 alone with that two-layer estimator: writes dk_out [B,C_a,3,3] fp32. */
int esc_convattn_dynkernel_mlp(const void* x, int B, int C, int C_a, int H, int W,
                               const void* w_down, const void* b_down,
                               const void* w_up, const void* b_up, int hidden, float* dk_out,
                               int dtype, int layout,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * Stage 1 for callers that must not allocate device memory.  (The paper has no counterpart:
 * this is a packaging variant of esc_convattn_dynkernel, same arithmetic, same result.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a real-time or
 * safety-certified loop whose memory is fixed at start-up, under an allocator-owning framework
 * that forbids side allocations, or in a process whose device memory is already fully handed
 * out.  Such callers cannot create the workspace the other entry points want, so here the
 * scratch (arrival counters and GAP partial sums) is a fixed 64 KiB array inside the library's
 * device image.  Every GPU that loads the library holds that array until the process exits.
 *
 *  - Limits: B <= 1024 and B * S * C_a <= 15360, where S (slabs per image) is 148 / B rounded down, at least 1
 *    (444 / B once B*H*W reaches 1.5 million pixels), capped at H*W/512.  Larger problems are
 *    refused with ESC_ERR_WORKSPACE and a message in esc_last_error(); nothing is enqueued.
 *  - The call itself allocates nothing: no cudaMalloc / cudaFree, no library allocator.  The very
 *    first call on each device looks up the array's device address (cudaGetSymbolAddress) with
 *    that device current; make that first call outside any stream capture.
 *  - All calls in the process share the one array.  The counters are cleared on `stream` at the
 *    start of every call; partial sums are overwritten before they are read.  Two calls whose GPU
 *    work overlaps (different streams, or different threads) race on it: serialise them.
 *  - Other arguments, layout rules, error codes and the result dk_out [B,C_a,3,3] fp32 are exactly
 *    those of esc_convattn_dynkernel.
 */
int esc_convattn_dynkernel_static(const void* x, int B, int C, int C_a, int H, int W,
                                  const void* w_dyn, const void* b_dyn, float* dk_out,
                                  int dtype, int layout, void* stream);

/*
 * Stage 2 alone (Eq. 4 lines 3-4 with an explicit dk [B,C_a,3,3] fp32 device array):
 * both depth-wise convolutions, their sum, and the copy of the remaining channels.
 * `workspace` may be NULL (then device-side time-outs cannot be reported).
 */
int esc_convattn_stencil(const void* x, int B, int C, int C_a, int H, int W, int K,
                         const void* w_large, const float* dk, void* out,
                         int dtype, int layout,
                         void* workspace, size_t workspace_bytes, void* stream);

/*
 * End-to-end convenience call on HOST buffers: copies x and the weights to the device,
 * runs the forward pass, copies out back and synchronises.  Device buffers and a private
 * stream are kept by the library between calls.  Host buffers should be pinned for full
 * copy bandwidth but need not be.
 */
int esc_convattn_forward_host(const void* x_host, int B, int C, int C_a, int H, int W, int K,
                              const void* w_large_host, const void* w_dyn_host,
                              const void* b_dyn_host, void* out_host, int dtype, int layout);

/*
 * The same end-to-end call split in two, so that a caller can keep the PCIe link busy in both
 * directions: submit enqueues the copies and the kernels on one of two private slots (slot 0 or 1,
 * each with its own device buffers and stream) and returns without waiting; wait blocks until that
 * slot's last submit has finished and out_host is complete.  With two slots in turn --
 * submit(i % 2) for step i, then wait((i - 1) % 2) -- the upload of one step overlaps the download
 * of the step before.  The host buffers must be pinned (page-locked) for the copies to be
 * asynchronous and must stay valid and untouched until the matching wait returns; two steps in
 * flight need two out_host buffers.  esc_convattn_forward_host is submit(0) followed by wait(0).
 * ESC_ERR_UNSUPPORTED for a slot other than 0 or 1.
 */
int esc_convattn_forward_host_submit(int slot, const void* x_host, int B, int C, int C_a, int H, int W, int K,
                                     const void* w_large_host, const void* w_dyn_host,
                                     const void* b_dyn_host, void* out_host, int dtype, int layout);
int esc_convattn_forward_host_wait(int slot);

/*
 * The decomposed large kernel of Eq. 5, F_res = (F_att (*) LK^c) (*) (ZP(DK) + LK^s): the attention
 * channels first go through the point-wise filter LK^c (a 1x1 convolution, no bias),
 *   w_point [C_a,C_a]   row n = output channel: mixed[n] = sum_k w_point[n,k] * F_att[k]
 * (device, the tensor's dtype), then through the same depth-wise stage as above; DK still comes from
 * GAP(F_att), the unmixed features (Eq. 4 line 2).  With bf16 storage the mixed features are rounded
 * to bf16 once where the fast kernel runs (NHWC, K = 13, C_a = 16: tensor-core mix inside the staged
 * tile) and kept in fp32 on the generic path.  Other arguments as for esc_convattn_forward_ex and
 * esc_convattn_stencil.
 */
int esc_convattn_forward_pw(const void* x, int B, int C, int C_a, int H, int W, int K,
                            const void* w_large, const void* w_point,
                            const void* w_dyn, const void* b_dyn,
                            void* out, int dtype, int layout,
                            void* workspace, size_t workspace_bytes, void* stream);

int esc_convattn_stencil_pw(const void* x, int B, int C, int C_a, int H, int W, int K,
                            const void* w_large, const void* w_point, const float* dk,
                            void* out, int dtype, int layout,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * The dense large kernel of the main ESC models (Section 3.2: LK in R^{13x13x16x16}) in Eq. 4 line 3:
 * every attention output channel sums over all C_a attention input channels and all K*K taps; the
 * dynamic 3x3 kernel stays depth-wise.
 *   w_dense [C_a,C_a,K,K]   (output channel, input channel, row, column), device, the tensor's dtype
 * For bf16 NHWC tensors with K = 13 and C_a = 16 the first sum runs on the tensor cores (bf16 products,
 * fp32 accumulation, implicit GEMM over the TMA-staged halo tile); anything else takes a slow
 * one-thread-per-output kernel.  Other arguments as for esc_convattn_forward_ex / esc_convattn_stencil.
 */
int esc_convattn_forward_dense(const void* x, int B, int C, int C_a, int H, int W, int K,
                               const void* w_dense, const void* w_dyn, const void* b_dyn,
                               void* out, int dtype, int layout,
                               void* workspace, size_t workspace_bytes, void* stream);

int esc_convattn_stencil_dense(const void* x, int B, int C, int C_a, int H, int W, int K,
                               const void* w_dense, const float* dk,
                               void* out, int dtype, int layout,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * Any combination of large-kernel form and estimator, i.e. the module as the paper's model variants use
 * it: ESC and ESC-light -- dense LK (Section 3.2) with the two-layer estimator, h = 8; ESC-FP -- the
 * decomposed LK of Eq. 5 with the two-layer estimator (Section 3.3 gives h = 4 or 8).
 *   large_kernel  ESC_LK_DEPTHWISE: w_large [C_a,K,K], w_point ignored
 *                 ESC_LK_DECOMPOSED: w_large [C_a,K,K] and w_point [C_a,C_a]
 *                 ESC_LK_DENSE: w_large [C_a,C_a,K,K], w_point ignored
 *   hidden        0: one linear layer, w_up [9*C_a,C_a] and b_up [9*C_a] play w_dyn and b_dyn, w_down and
 *                 b_down are ignored; 1..128: the two-layer estimator with the exact GELU
 * Everything else as for esc_convattn_forward_ex.  ESC_ERR_UNSUPPORTED for an unknown large_kernel.
 */
enum { ESC_LK_DEPTHWISE = 0, ESC_LK_DECOMPOSED = 1, ESC_LK_DENSE = 2 };
int esc_convattn_forward_variant(const void* x, int B, int C, int C_a, int H, int W, int K, int large_kernel,
                                 const void* w_large, const void* w_point,
                                 const void* w_down, const void* b_down,
                                 const void* w_up, const void* b_up, int hidden,
                                 void* out, int dtype, int layout,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* The whole module including its last step (Section 3.3, Eq. 4 lines 1-4) and the residual connection of the ESC
 * block around it (Eq. 3 line 3), for the depth-wise large kernel with the one-layer estimator:
 *   cat = esc_convattn_forward_ex(x)                                   (F_res | F_idt)
 *   out[b,n,y,x] = b_fuse[n] + sum_c w_fuse[n,c] * cat[b,c,y,x]  ( + residual[b,n,y,x] )
 *   w_fuse     [C,C]        same dtype as x, row = output channel (Conv_fuse, 1x1)
 *   b_fuse     [C]          same dtype, may be NULL
 *   residual   [B,C,H,W]    same dtype and layout as x, 16-byte aligned, may be NULL, may be x itself; must not overlap out
 * Everything else as for esc_convattn_forward_ex.  Asynchronous on `stream`.
 * NHWC bf16 with C in {32, 48, 64, 96, 128}, C_a a multiple of 16, K = 13 and 16-byte aligned w_fuse: the stencil kernel
 * writes only the attention channels, and a tensor-core 1x1 kernel reads them back together with the identity channels
 * straight from x -- the concatenation is never copied (2 or 3 launches).  F_res passes through out as bf16 there, so it
 * is rounded once before Conv_fuse, as it would be between two layers of a bf16 network; all sums are fp32 and the result
 * is rounded once.  Every other configuration runs esc_convattn_forward_ex into out and a guarded 1x1 kernel in place
 * (C * 128 bytes of shared memory per block: ESC_ERR_UNSUPPORTED beyond C = 384). */
int esc_convattn_forward_fused(const void* x, int B, int C, int C_a, int H, int W, int K,
                               const void* w_large, const void* w_dyn, const void* b_dyn,
                               const void* w_fuse, const void* b_fuse, const void* residual,
                               void* out, int dtype, int layout,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass of esc_convattn_forward_ex (one-layer estimator, depth-wise LK; the chain rule applied to
 * Eq. 4): given grad_out = dL/dout, writes
 *   grad_x        [B,C,H,W]    dL/dx, element type and layout of x (identity channels: grad_out itself; attention
 *                              channels: grad_out correlated with the 180-degree-rotated merged kernels, plus the
 *                              path through the GAP and the estimator)
 *   grad_w_large  [C_a,K,K]    fp32   dL/dLK        (may be NULL)
 *   grad_w_dyn    [9*C_a,C_a]  fp32   dL/dW_dyn     (may be NULL)
 *   grad_b_dyn    [9*C_a]      fp32   dL/db_dyn     (may be NULL)
 * K must be odd, 3 .. 13 (ESC_ERR_UNSUPPORTED above 13).  grad_x must not overlap x or grad_out.  The workspace is one of
 * esc_convattn_backward_workspace_bytes(...) bytes, 256-byte aligned, zeroed once with
 * esc_convattn_workspace_init(); it is not the forward workspace.  All sums are added in a fixed order.
 */
size_t esc_convattn_backward_workspace_bytes(int B, int C_a, int H, int W, int K);
int esc_convattn_backward(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                          const void* w_large, const void* w_dyn, const void* b_dyn,
                          void* grad_x, float* grad_w_large, float* grad_w_dyn, float* grad_b_dyn,
                          int dtype, int layout,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass of esc_convattn_forward_mlp: the same with the estimator as Eq. 4 line 2 writes it,
 * dk = W_up phi(W_down g + b_down) + b_up with phi(t) = t Phi(t) (exact GELU), differentiated through
 * phi'(t) = Phi(t) + t n(t) (n the standard normal density).  Weight layouts as in esc_convattn_forward_mlp:
 * w_down [hidden,C_a], b_down [hidden], w_up [9*C_a,hidden], b_up [9*C_a], element type of x; 1 <= hidden <= 128.
 *   grad_x        [B,C,H,W]        as above
 *   grad_w_large  [C_a,K,K]        fp32   (may be NULL)
 *   grad_w_down   [hidden,C_a]     fp32   (may be NULL)        grad_b_down [hidden]   fp32 (may be NULL)
 *   grad_w_up     [9*C_a,hidden]   fp32   (may be NULL)        grad_b_up   [9*C_a]    fp32 (may be NULL)
 * Same workspace, restrictions and error codes as esc_convattn_backward; ESC_ERR_SHAPE for hidden out of range.
 */
int esc_convattn_backward_mlp(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                              const void* w_large, const void* w_down, const void* b_down,
                              const void* w_up, const void* b_up, int hidden,
                              void* grad_x, float* grad_w_large, float* grad_w_down, float* grad_b_down,
                              float* grad_w_up, float* grad_b_up, int dtype, int layout,
                              void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass of esc_convattn_forward_pw, the decomposed form of Eq. 5: the point-wise filter LK^c (w_point [C_a,C_a],
 * row = output channel, element type of x) in front of the depth-wise stage, one-layer estimator fed by the GAP of the
 * unmixed features.  With m = LK^c x_att and g_m = dL/dm (grad_out through the rotated depth-wise kernels):
 *   grad_w_point [C_a,C_a]  fp32   dL/dLK^c[n,k] = sum over images and pixels of g_m[n] x[k]   (may be NULL)
 *   grad_x attention channels = LK^c transposed applied to g_m, plus the estimator's path; identity channels = grad_out
 *   grad_w_large, grad_w_dyn, grad_b_dyn as in esc_convattn_backward, with m in the place of x_att (grad_w_dyn still
 *   multiplies the mean of the unmixed features).
 * m and g_m are kept in the element type of x (one rounding each for bf16), in grad_x's attention channels, so grad_x
 * is also scratch while the call runs.  C_a must be 4, 8, 16 or 32 (ESC_ERR_UNSUPPORTED otherwise).  Same workspace,
 * restrictions and error codes as esc_convattn_backward.  All device memory; asynchronous on `stream`.
 */
int esc_convattn_backward_pw(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                             const void* w_large, const void* w_point, const void* w_dyn, const void* b_dyn,
                             void* grad_x, float* grad_w_large, float* grad_w_point, float* grad_w_dyn,
                             float* grad_b_dyn, int dtype, int layout,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass of esc_convattn_forward_dense, the dense large kernel of Section 3.2 (w_dense [C_a,C_a,K,K]: output
 * channel, input channel, row, column; element type of x), depth-wise dynamic kernel, one-layer estimator:
 *   grad_w_dense [C_a,C_a,K,K]  fp32   dL/dw_dense[n,k,i,j] = sum over images and pixels of grad_out[n,y,x] x~[k,y+i-P,x+j-P]  (may be NULL)
 *   grad_x, grad_w_dyn, grad_b_dyn as in esc_convattn_backward (grad_x's large-kernel term sums over the output channels).
 * C_a must be 16 (ESC_ERR_UNSUPPORTED otherwise); K odd, 3 .. 13.  The workspace is one of
 * esc_convattn_backward_dense_workspace_bytes(...) bytes (larger than the depth-wise one: every block of the tap-gradient
 * kernel keeps 16 x 16 x 169 sums there), 256-byte aligned, zeroed once with esc_convattn_workspace_init().  Same
 * restrictions and error codes as esc_convattn_backward.  All device memory; asynchronous on `stream`.
 */
size_t esc_convattn_backward_dense_workspace_bytes(int B, int C_a, int H, int W, int K);
int esc_convattn_backward_dense(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                                const void* w_dense, const void* w_dyn, const void* b_dyn,
                                void* grad_x, float* grad_w_dense, float* grad_w_dyn, float* grad_b_dyn,
                                int dtype, int layout,
                                void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass of esc_convattn_forward_variant: any large-kernel form (ESC_LK_*) with either estimator -- the
 * configurations the paper's models use are the dense and the decomposed large kernel with the two-layer estimator of
 * Eq. 4 line 2.  Arguments as in esc_convattn_forward_variant (hidden = 0: one linear layer w_up [9*C_a,C_a], b_up; w_down,
 * b_down and their gradients ignored), gradients as in esc_convattn_backward_mlp, _pw and _dense:
 *   grad_w_large  [C_a,K,K], or [C_a,C_a,K,K] for ESC_LK_DENSE   fp32 (may be NULL)
 *   grad_w_point  [C_a,C_a] for ESC_LK_DECOMPOSED                 fp32 (may be NULL; ignored otherwise)
 *   grad_w_down [hidden,C_a], grad_b_down [hidden], grad_w_up [9*C_a,hidden or C_a], grad_b_up [9*C_a]   fp32 (may be NULL)
 * Restrictions of the form's own entry apply (ESC_LK_DECOMPOSED: C_a 4, 8, 16 or 32; ESC_LK_DENSE: C_a = 16 and the
 * workspace of esc_convattn_backward_dense_workspace_bytes; otherwise esc_convattn_backward_workspace_bytes).
 */
int esc_convattn_backward_variant(const void* x, const void* grad_out, int B, int C, int C_a, int H, int W, int K,
                                  int large_kernel, const void* w_large, const void* w_point, const void* w_down,
                                  const void* b_down, const void* w_up, const void* b_up, int hidden, void* grad_x,
                                  float* grad_w_large, float* grad_w_point, float* grad_w_down, float* grad_b_down,
                                  float* grad_w_up, float* grad_b_up, int dtype, int layout,
                                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass of the module's closing 1x1 convolution with the block's residual (Eq. 4 line 4, Eq. 3 line 3:
 * out = W_fuse cat + b_fuse + residual per pixel; what esc_convattn_forward_fused adds behind the ConvAttn stages).
 *   cat           [B,C,H,W]  the convolution's input (the concatenated map, i.e. esc_convattn_forward's output), device
 *   grad_out      [B,C,H,W]  dL/dout, element type and layout of cat; it is also the residual's gradient
 *   grad_cat      [B,C,H,W]  written: W_fuse transposed applied to grad_out -- the grad_out of esc_convattn_backward*
 *   grad_w_fuse   [C,C] fp32  sum over images and pixels of grad_out[n] cat[c]   (may be NULL)
 *   grad_b_fuse   [C]   fp32  sum over images and pixels of grad_out[n]          (may be NULL)
 * C must be 16, 32, 48 or 64 (ESC_ERR_UNSUPPORTED otherwise).  grad_cat must not overlap cat or grad_out.  The workspace
 * is one of esc_conv_fuse_backward_workspace_bytes(...) bytes, 256-byte aligned; it needs no initialisation.  All sums
 * are added in a fixed order.  All device memory; asynchronous on `stream`.
 */
size_t esc_conv_fuse_backward_workspace_bytes(int B, int C, int H, int W);
int esc_conv_fuse_backward(const void* cat, const void* grad_out, int B, int C, int H, int W, const void* w_fuse,
                           void* grad_cat, float* grad_w_fuse, float* grad_b_fuse, int dtype, int layout,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Self-test of the error path that every device-side wait of this library shares: launches one thread that waits, with
 * the kernels' own bounded wait, on a barrier that nothing signals.  The wait gives up after its poll limit (about one
 * second), records ESC_DEV_TIMEOUT in the status word of `workspace` (any initialised forward or backward workspace, device)
 * and the kernel returns normally: no trap, no fault, the context stays usable.  esc_convattn_device_status() then returns
 * ESC_DEV_TIMEOUT once and clears the word.  Asynchronous on `stream`.
 */
int esc_convattn_selftest_bounded_wait(void* workspace, void* stream);

/* Synchronises `stream`, returns the workspace status word (ESC_OK or ESC_DEV_TIMEOUT) and
 * clears it. */
int esc_convattn_device_status(void* workspace, void* stream);

/* Which stencil implementation the last esc_convattn_forward* / esc_convattn_stencil call on
 * this thread selected: 0 = none yet, 1 = guarded generic kernel, 2 = TMA-staged register-tiled
 * FP32 kernel, 3 = tensor-core kernel of the dense large kernel, 4 = tensor-core (banded Toeplitz)
 * kernel of the depth-wise large kernel on NHWC tensors, 5 = tcgen05 kernel of the dense large kernel,
 * 6 = the tensor-core (banded Toeplitz) kernel on NCHW tensors.  For tests and benchmarks. */
int esc_convattn_last_path(void);

/* Which arithmetic units evaluate the depth-wise large-kernel stage of Eq. 4 line 3 on bf16 tensors (and the tap
 * gradients of the backward pass), for later calls on this thread.  ESC_ENGINE_AUTO (default): the tensor-core
 * kernels where they apply -- odd K up to 13 (a smaller kernel is zero-padded to 13 x 13 in the workspace), C_a a
 * multiple of 16; NHWC with C a multiple of 8 (also with the point-wise LK^c when C_a = 16), or NCHW with W a
 * multiple of 8 and 16-byte aligned tensors -- else the FP32 kernels.
 * ESC_ENGINE_FP32: never the tensor-core kernel.  ESC_ENGINE_TENSOR: the tensor-core kernel or, where
 * it does not apply, the guarded generic kernel.  Both engines multiply exactly (bf16 x bf16 in fp32) and
 * accumulate in fp32; they differ in the order of the 169 additions, i.e. by fp32 rounding before
 * the single rounding of the result to bf16.  In the tensor-core kernel one instruction sums 16
 * horizontally adjacent inputs, three of which may lie outside an output's 13-tap window with weight
 * zero: a non-finite attention input therefore turns outputs up to 15 pixels beyond its window into
 * NaN (finite data are unaffected).  Returns ESC_ERR_UNSUPPORTED for any other value. */
enum { ESC_ENGINE_AUTO = 0, ESC_ENGINE_FP32 = 1, ESC_ENGINE_TENSOR = 2 };
int esc_convattn_set_stencil_engine(int engine);

/* Whether a forward call on this thread may run as ONE launch of the tensor-core kernel with stage 1 (Eq. 4
 * line 2: pooled means and the kernel estimator) inside it (default: on).  It does so where that kernel applies,
 * C_a <= 128, and no CTA gets more than two 64x16 tiles (about 300,000 pixels per 16 attention channels on a
 * B200): every CTA adds up the interiors of its own staged tiles, the CTAs exchange the sums through the
 * workspace and each evaluates the estimator for the channels it works on.  The launch is cooperative (CTAs
 * wait on one another, all waits bounded: ESC_DEV_TIMEOUT through esc_convattn_device_status); if the device
 * refuses it, or with 0 here, the forward is the usual two launches.  The pooled means are then sums over tiles
 * instead of slabs: dk differs by fp32 rounding (about 1e-7 relative).  A workspace whose launch was cut short
 * must be zeroed again with esc_convattn_workspace_init before its next use.  For tests and tuning. */
int esc_convattn_set_fused_stage1(int on);

/* Which kernel evaluates the dense large kernel of Section 3.2 (esc_convattn_forward_dense / _stencil_dense /
 * ESC_LK_DENSE) on NHWC bf16 tensors with 16 attention channels and K = 13, for later calls on this thread:
 * 0 (default) = the tcgen05 kernel (accumulators in tensor memory, one instruction per input row and tap column
 * with all 13 kernel rows stacked in N), 1 = the warp-level mma.sync kernel.  Both multiply exactly and accumulate
 * in fp32; they differ in the order of the additions.  esc_convattn_last_path() reports 5 and 3.  Returns
 * ESC_ERR_UNSUPPORTED for any other value.  For tests and comparisons. */
int esc_convattn_set_dense_engine(int engine);

/* Width in pixels of the output tile the TMA-staged kernel used in that call (FP32 kernel: 40 = 40x40
 * tiles, 64 = 64x16 tiles, chosen by the tile count's balance over the SMs; tensor-core kernel: 64 =
 * 64x16 tiles), 0 when the generic kernel ran.  For tests and benchmarks. */
int esc_convattn_last_tile_width(void);

/* Overrides the tile choice of the TMA-staged FP32 kernel for later calls on this thread (and, when
 * not 0, selects that kernel as ESC_ENGINE_FP32 does): 0 = choose by cost (the default), 40 or 64 =
 * always that width.  The geometries add the 169 taps of an
 * output in different orders, so results differ by fp32 rounding before the final rounding to
 * bf16 (far inside the module's tolerance); with a fixed width, results are bitwise reproducible.
 * Returns ESC_ERR_UNSUPPORTED for any other value.  For tests and tuning. */
int esc_convattn_set_tile_width(int tile_width);

/* Number of kernels the last forward / stage call on this thread launched. */
int esc_convattn_last_launches(void);

const char* esc_status_string(int status);
const char* esc_last_error(void);   /* thread-local text of the last ESC_ERR_CUDA */
int esc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ESC_CONVATTN_H */

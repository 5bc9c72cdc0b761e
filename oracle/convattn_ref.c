/*
 * TEST INFRASTRUCTURE -- CPU oracle for the ConvAttn forward pass.
 *
 * This file is the slow, obviously-correct definition that the CUDA library is
 * checked against.  It is used only by the test-suite, by the smoke check and
 * by the benchmark's CPU-baseline leg; the product never calls it and it shares
 * no code, header, table or helper with the CUDA path.
 *
 * What it computes (ESC paper, Section 3.3 "Convolutional Attention Module",
 * Eq. 4, in the depth-wise form of Eq. 5 without the point-wise LK^c, and with
 * the kernel estimator reduced to one linear layer):
 *
 *   F_att = x[:, :C_a],  F_idt = x[:, C_a:]                      (Eq. 4, line 1)
 *   g[b,c]   = mean over (y,x) of F_att[b,c,y,x]                 (GAP, Eq. 4 line 2)
 *   dk[b,o]  = b_dyn[o] + sum_c W_dyn[o,c] * g[b,c],  o = c*9+i*3+j
 *   out[b,c] = F_att[b,c] (*) LK[c]  +  F_att[b,c] (*) dk[b,c]   (Eq. 4, line 3)
 *   out[b, C_a:] = F_idt                                         (Concat, Eq. 4 line 4)
 *
 * convattn_ref_dynkernel_mlp is the estimator exactly as Eq. 4 line 2 writes it,
 *   dk[b] = W_up . phi(W_down . g[b] + b_down) + b_up,   phi(t) = t * Phi(t)   (GELU, exact erf form)
 * with hidden width h; the other stages are shared.
 *
 * convattn_ref_pointwise + convattn_ref_stencil_mixed are the decomposed form of Eq. 5,
 *   out[b,:C_a] = (F_att (*) LK^c) (*) (ZP(dk) + LK^s),  LK^c a 1x1 convolution over the C_a channels,
 * taken in that order: mix first, then the depth-wise stage on the mixed features; dk still
 * comes from GAP(F_att) as in Eq. 4 line 2.
 *
 * convattn_ref_stencil_dense is Eq. 4 line 3 with the dense large kernel of Section 3.2
 * (13x13x16x16: every output channel sums over all attention input channels).
 *
 * convattn_ref_fuse is the module's last step, Conv_fuse over the concatenated channels (Eq. 4 line 4),
 * with the block's residual connection (Eq. 3 line 3).
 *
 * convattn_ref_backward is the gradient of the first form above with respect to x, LK, W_dyn and
 * b_dyn, by the chain rule written out; convattn_ref_backward_mlp the same with the two-layer estimator
 * (gradients with respect to x, LK, W_down, b_down, W_up, b_up).
 * convattn_ref_backward_pw is the gradient of the decomposed form (x, LK^s, LK^c, W_dyn, b_dyn).
 * convattn_ref_backward_dense is the gradient of the dense form (x, the dense LK, W_dyn, b_dyn).
 *
 * (*) is cross-correlation (no kernel flip) with zero 'same' padding.
 * Everything is accumulated in double precision with direct nested loops in
 * the order written above: no tiling, no merging of the two kernels, no reuse.
 * Inputs are float arrays holding exactly the values the device sees (bf16
 * values widen to float without change); weights are passed as double.
 *
 * OpenMP only spreads independent (image, channel, row) iterations over
 * threads for the timing harness; every output value is produced by exactly the
 * same sequence of operations whatever the thread count.
 *
 * Pinned by tests/test_oracle_pins.py (impulse response, constant-input closed
 * form, zero generator vs a library convolution, scatter-form brute force on
 * tiny inputs, linearity laws, the Eq. 5 merge identity, permutation / batch
 * independence, and the GAP->dk stage on non-zero-mean data); the two-layer
 * estimator by tabulated values of the normal distribution function, the
 * reflection law of phi, its two linear limits (which reduce it to the one-layer
 * estimator with composed weights) and a math.erf brute force; the decomposed form
 * by the identity mix, library 1x1 + depth-wise convolutions, the commutation with a
 * channel-independent spatial kernel, permutation mixes and a brute force; the dense
 * large kernel by its diagonal case (= the depth-wise stencil), a library dense
 * convolution, the depth-wise-then-point-wise factorisation and a brute force; the
 * backward pass by central differences of the pinned forward (exact for this
 * function, which is quadratic in x and bilinear in weights and x) and the
 * adjoint identity; the backward pass with the two-layer estimator by central differences of
 * the pinned forward and by its linear limit, where it must equal the pinned one-layer backward
 * with composed weights; the backward pass of the decomposed form by central differences of the pinned
 * decomposed forward (also exact), by the identity mix, where it must equal the pinned depth-wise backward,
 * and by the adjoint identity of its linear part; the backward pass with the dense large kernel by exact
 * differences of the pinned dense forward and by its diagonal case, where it must equal the pinned depth-wise
 * backward; the backward pass of Conv_fuse by exact differences of the pinned convattn_ref_fuse (linear in its
 * input and in each weight) and by the identity matrix.
 */
#include <stddef.h>
#include <stdint.h>
#include <math.h>
#include <stdlib.h>

#define IDX4(b, c, y, x, C, H, W) ((((size_t)(b) * (C) + (c)) * (H) + (y)) * (size_t)(W) + (x))

/* GAP over the first C_a channels of x[B,C,H,W] (Eq. 4, line 2, inner term). g is [B,C_a]. */
void convattn_ref_gap(const float *x, int B, int C, int C_a, int H, int W, double *g)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C_a; ++c) {
            double s = 0.0;
            for (int y = 0; y < H; ++y)
                for (int xx = 0; xx < W; ++xx)
                    s += (double)x[IDX4(b, c, y, xx, C, H, W)];
            g[(size_t)b * C_a + c] = s / ((double)H * (double)W);
        }
}

/* Kernel estimator: one linear layer C_a -> 9*C_a with bias. dk is [B, C_a*9],
 * output index o = c*9 + i*3 + j holds tap (i,j) of channel c's 3x3 kernel. */
void convattn_ref_dynkernel(const double *g, int B, int C_a, const double *w_dyn, const double *b_dyn,
                            double *dk)
{
    for (int b = 0; b < B; ++b)
        for (int o = 0; o < 9 * C_a; ++o) {
            double s = b_dyn[o];
            for (int c = 0; c < C_a; ++c)
                s += w_dyn[(size_t)o * C_a + c] * g[(size_t)b * C_a + c];
            dk[(size_t)b * 9 * C_a + o] = s;
        }
}

/* Gaussian error linear unit: phi(t) = t * Phi(t), Phi the standard normal distribution function,
 * Phi(t) = (1 + erf(t / sqrt 2)) / 2 = erfc(-t / sqrt 2) / 2; the erfc form keeps full relative
 * accuracy in the left tail, where 1 + erf cancels. */
static double gelu(double t)
{
    return t * 0.5 * erfc(-t / sqrt(2.0));
}

/* Kernel estimator of Eq. 4 line 2: Conv_up(phi(Conv_down(g))), both 1x1 convolutions on a 1x1 map, i.e.
 * two dense layers with bias.  w_down [h, C_a], b_down [h], w_up [9*C_a, h], b_up [9*C_a]; hidden (may be
 * NULL) receives phi(...) [B, h]; dk is [B, C_a*9] with the same output order as the one-layer estimator. */
void convattn_ref_dynkernel_mlp(const double *g, int B, int C_a, int h, const double *w_down,
                                const double *b_down, const double *w_up, const double *b_up,
                                double *hidden, double *dk)
{
    for (int b = 0; b < B; ++b) {
        double a[256];                       /* h <= 256, checked by the caller */
        for (int j = 0; j < h; ++j) {
            double t = b_down[j];
            for (int c = 0; c < C_a; ++c)
                t += w_down[(size_t)j * C_a + c] * g[(size_t)b * C_a + c];
            a[j] = gelu(t);
            if (hidden) hidden[(size_t)b * h + j] = a[j];
        }
        for (int o = 0; o < 9 * C_a; ++o) {
            double s = b_up[o];
            for (int j = 0; j < h; ++j)
                s += w_up[(size_t)o * h + j] * a[j];
            dk[(size_t)b * 9 * C_a + o] = s;
        }
    }
}

/* One output value of an attention channel (c < C_a): large-kernel taps, then the
 * dynamic 3x3 taps, both with zero padding.  *mag receives sum |w * x| over the
 * same taps (the scale that bounds the rounding error of any evaluation order). */
static double one_output(const float *x, int C, int H, int W, int K, const double *w_large,
                         const double *dk_b, int b, int c, int y, int xx, double *mag)
{
    const int P = (K - 1) / 2;
    double s = 0.0, m = 0.0;
    for (int i = 0; i < K; ++i)
        for (int j = 0; j < K; ++j) {
            int yy = y + i - P, xc = xx + j - P;
            if (yy >= 0 && yy < H && xc >= 0 && xc < W) {
                double t = w_large[((size_t)c * K + i) * K + j] * (double)x[IDX4(b, c, yy, xc, C, H, W)];
                s += t;
                m += fabs(t);
            }
        }
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) {
            int yy = y + i - 1, xc = xx + j - 1;
            if (yy >= 0 && yy < H && xc >= 0 && xc < W) {
                double t = dk_b[c * 9 + i * 3 + j] * (double)x[IDX4(b, c, yy, xc, C, H, W)];
                s += t;
                m += fabs(t);
            }
        }
    if (mag) *mag = m;
    return s;
}

/* Stencil stage with an explicit dk[B,C_a*9]: rows y0..y1-1 of every image.
 * out is [B, C, y1-y0, W] (attention channels convolved, the others copied);
 * mag (optional, may be NULL) is [B, C_a, y1-y0, W]. */
void convattn_ref_stencil(const float *x, int B, int C, int C_a, int H, int W, int K,
                          const double *w_large, const double *dk, int y0, int y1, double *out,
                          double *mag)
{
    const int R = y1 - y0;
#pragma omp parallel for collapse(3) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C; ++c)
            for (int y = y0; y < y1; ++y) {
                for (int xx = 0; xx < W; ++xx) {
                    size_t o = IDX4(b, c, y - y0, xx, C, R, W);
                    if (c < C_a) {
                        double m;
                        out[o] = one_output(x, C, H, W, K, w_large, dk + (size_t)b * 9 * C_a, b, c, y, xx, &m);
                        if (mag) mag[IDX4(b, c, y - y0, xx, C_a, R, W)] = m;
                    } else {
                        out[o] = (double)x[IDX4(b, c, y, xx, C, H, W)];
                    }
                }
            }
}

/* Whole forward pass. g_out [B,C_a] and dk_out [B,C_a*9] are scratch the caller
 * provides and may inspect; mag may be NULL. */
void convattn_ref_forward(const float *x, int B, int C, int C_a, int H, int W, int K,
                          const double *w_large, const double *w_dyn, const double *b_dyn,
                          double *out, double *g_out, double *dk_out, double *mag)
{
    convattn_ref_gap(x, B, C, C_a, H, W, g_out);
    convattn_ref_dynkernel(g_out, B, C_a, w_dyn, b_dyn, dk_out);
    convattn_ref_stencil(x, B, C, C_a, H, W, K, w_large, dk_out, 0, H, out, mag);
}

/* The module's last step (Eq. 4 line 4): F_fuse = Conv_fuse(Concat(F_res, F_idt)), a 1x1 convolution over all C
 * channels of the concatenated map `cat` [B,C,H,W] (the output of the stages above), with bias, and the residual
 * connection of the ESC block around the module (Eq. 3 line 3: F_{i,j} = F_{i,j-1} + ConvAttn(...)):
 *   out[b,n,y,x] = b_fuse[n] + sum_c w_fuse[n,c] * cat[b,c,y,x]  ( + residual[b,n,y,x] )
 * b_fuse and residual may be NULL.  mag (optional) [B,C,H,W] receives |b_fuse[n]| + sum_c |w_fuse[n,c] * cat| + |residual|. */
void convattn_ref_fuse(const double *cat, int B, int C, int H, int W, const double *w_fuse, const double *b_fuse,
                       const float *residual, double *out, double *mag)
{
#pragma omp parallel for collapse(3) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < C; ++n)
            for (int y = 0; y < H; ++y)
                for (int xx = 0; xx < W; ++xx) {
                    double s = b_fuse ? b_fuse[n] : 0.0, m = fabs(s);
                    for (int c = 0; c < C; ++c) {
                        double t = w_fuse[(size_t)n * C + c] * cat[IDX4(b, c, y, xx, C, H, W)];
                        s += t;
                        m += fabs(t);
                    }
                    if (residual) {
                        double r = (double)residual[IDX4(b, n, y, xx, C, H, W)];
                        s += r;
                        m += fabs(r);
                    }
                    out[IDX4(b, n, y, xx, C, H, W)] = s;
                    if (mag) mag[IDX4(b, n, y, xx, C, H, W)] = m;
                }
}

/* Backward pass of convattn_ref_fuse.  With go = dL/dout [B,C,H,W] (float values) and cat the forward's input:
 *   g_cat[b,c,y,x] = sum_n w_fuse[n,c] * go[b,n,y,x]
 *   g_w[n,c]       = sum_{b,y,x} go[b,n,y,x] * cat[b,c,y,x]
 *   g_b[n]         = sum_{b,y,x} go[b,n,y,x]
 * (the residual's gradient is go itself).  mag_cat (optional) receives sum_n |w_fuse[n,c] * go|; any output may be NULL. */
void convattn_ref_fuse_backward(const float *cat, const float *go, int B, int C, int H, int W, const double *w_fuse,
                                double *g_cat, double *g_w, double *g_b, double *mag_cat)
{
    if (g_cat) {
#pragma omp parallel for collapse(3) schedule(static)
        for (int b = 0; b < B; ++b)
            for (int c = 0; c < C; ++c)
                for (int y = 0; y < H; ++y)
                    for (int xx = 0; xx < W; ++xx) {
                        double s = 0.0, m = 0.0;
                        for (int n = 0; n < C; ++n) {
                            double t = w_fuse[(size_t)n * C + c] * (double)go[IDX4(b, n, y, xx, C, H, W)];
                            s += t;
                            m += fabs(t);
                        }
                        g_cat[IDX4(b, c, y, xx, C, H, W)] = s;
                        if (mag_cat) mag_cat[IDX4(b, c, y, xx, C, H, W)] = m;
                    }
    }
    if (g_w) {
#pragma omp parallel for collapse(2) schedule(static)
        for (int n = 0; n < C; ++n)
            for (int c = 0; c < C; ++c) {
                double s = 0.0;
                for (int b = 0; b < B; ++b)
                    for (int y = 0; y < H; ++y)
                        for (int xx = 0; xx < W; ++xx)
                            s += (double)go[IDX4(b, n, y, xx, C, H, W)] * (double)cat[IDX4(b, c, y, xx, C, H, W)];
                g_w[(size_t)n * C + c] = s;
            }
    }
    if (g_b)
        for (int n = 0; n < C; ++n) {
            double s = 0.0;
            for (int b = 0; b < B; ++b)
                for (int y = 0; y < H; ++y)
                    for (int xx = 0; xx < W; ++xx) s += (double)go[IDX4(b, n, y, xx, C, H, W)];
            g_b[n] = s;
        }
}

/* Point-wise large-kernel filter LK^c of the decomposed form (Eq. 5, first factor F_att (*) LK^c):
 * a 1x1 convolution over the attention channels, no bias.
 *   xm[b,n,y,x] = sum_k w_point[n,k] * x[b,k,y,x]        n, k < C_a
 * xm is [B, C_a, H, W]; xabs (optional) receives sum_k |w_point[n,k] * x[b,k,y,x]|. */
void convattn_ref_pointwise(const float *x, int B, int C, int C_a, int H, int W, const double *w_point,
                            double *xm, double *xabs)
{
#pragma omp parallel for collapse(3) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < C_a; ++n)
            for (int y = 0; y < H; ++y)
                for (int xx = 0; xx < W; ++xx) {
                    double s = 0.0, m = 0.0;
                    for (int k = 0; k < C_a; ++k) {
                        double t = w_point[(size_t)n * C_a + k] * (double)x[IDX4(b, k, y, xx, C, H, W)];
                        s += t;
                        m += fabs(t);
                    }
                    xm[IDX4(b, n, y, xx, C_a, H, W)] = s;
                    if (xabs) xabs[IDX4(b, n, y, xx, C_a, H, W)] = m;
                }
}

/* Eq. 5, second factor: the mixed features xm [B,C_a,H,W] convolved depth-wise with LK^s and with
 * the dynamic 3x3 kernel (the two convolutions of Eq. 4 line 3, summed; same taps as ZP(DK) + LK^s),
 * zero padding; identity channels copied from x.  out is [B,C,H,W]; mag (optional) [B,C_a,H,W]
 * receives sum |w| * xabs over the same taps when xabs is given, else sum |w * xm|. */
void convattn_ref_stencil_mixed(const float *x, const double *xm, const double *xabs, int B, int C, int C_a,
                                int H, int W, int K, const double *w_large, const double *dk, double *out,
                                double *mag)
{
    const int P = (K - 1) / 2;
#pragma omp parallel for collapse(3) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C; ++c)
            for (int y = 0; y < H; ++y)
                for (int xx = 0; xx < W; ++xx) {
                    if (c >= C_a) {
                        out[IDX4(b, c, y, xx, C, H, W)] = (double)x[IDX4(b, c, y, xx, C, H, W)];
                        continue;
                    }
                    double s = 0.0, m = 0.0;
                    for (int i = 0; i < K; ++i)
                        for (int j = 0; j < K; ++j) {
                            int yy = y + i - P, xc = xx + j - P;
                            if (yy >= 0 && yy < H && xc >= 0 && xc < W) {
                                size_t q = IDX4(b, c, yy, xc, C_a, H, W);
                                double w = w_large[((size_t)c * K + i) * K + j];
                                s += w * xm[q];
                                m += fabs(w) * (xabs ? xabs[q] : fabs(xm[q]));
                            }
                        }
                    for (int i = 0; i < 3; ++i)
                        for (int j = 0; j < 3; ++j) {
                            int yy = y + i - 1, xc = xx + j - 1;
                            if (yy >= 0 && yy < H && xc >= 0 && xc < W) {
                                size_t q = IDX4(b, c, yy, xc, C_a, H, W);
                                double w = dk[(size_t)b * 9 * C_a + c * 9 + i * 3 + j];
                                s += w * xm[q];
                                m += fabs(w) * (xabs ? xabs[q] : fabs(xm[q]));
                            }
                        }
                    out[IDX4(b, c, y, xx, C, H, W)] = s;
                    if (mag) mag[IDX4(b, c, y, xx, C_a, H, W)] = m;
                }
}

/* Dense large kernel (Section 3.2: LK in R^{13x13x16x16}; Eq. 4 line 3 with that LK): every attention
 * output channel n sums over all C_a input channels k and all taps,
 *   out[b,n,y,x] = sum_{k,i,j} w_dense[n,k,i,j] * x[b,k,y+i-P,x+j-P]  +  sum_{i,j} dk[b,n,i,j] * x[b,n,y+i-1,x+j-1],
 * zero padding, the dynamic 3x3 kernel still depth-wise; identity channels copied.  w_dense is
 * [C_a, C_a, K, K] (output channel, input channel, row, column); out [B,C,H,W]; mag (optional) [B,C_a,H,W]
 * receives sum |w * x| over the same terms. */
void convattn_ref_stencil_dense(const float *x, int B, int C, int C_a, int H, int W, int K,
                                const double *w_dense, const double *dk, double *out, double *mag)
{
    const int P = (K - 1) / 2;
#pragma omp parallel for collapse(3) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < C; ++n)
            for (int y = 0; y < H; ++y)
                for (int xx = 0; xx < W; ++xx) {
                    if (n >= C_a) {
                        out[IDX4(b, n, y, xx, C, H, W)] = (double)x[IDX4(b, n, y, xx, C, H, W)];
                        continue;
                    }
                    double s = 0.0, m = 0.0;
                    for (int k = 0; k < C_a; ++k)
                        for (int i = 0; i < K; ++i)
                            for (int j = 0; j < K; ++j) {
                                int yy = y + i - P, xc = xx + j - P;
                                if (yy >= 0 && yy < H && xc >= 0 && xc < W) {
                                    double t = w_dense[(((size_t)n * C_a + k) * K + i) * K + j] *
                                               (double)x[IDX4(b, k, yy, xc, C, H, W)];
                                    s += t;
                                    m += fabs(t);
                                }
                            }
                    for (int i = 0; i < 3; ++i)
                        for (int j = 0; j < 3; ++j) {
                            int yy = y + i - 1, xc = xx + j - 1;
                            if (yy >= 0 && yy < H && xc >= 0 && xc < W) {
                                double t = dk[(size_t)b * 9 * C_a + n * 9 + i * 3 + j] * (double)x[IDX4(b, n, yy, xc, C, H, W)];
                                s += t;
                                m += fabs(t);
                            }
                        }
                    out[IDX4(b, n, y, xx, C, H, W)] = s;
                    if (mag) mag[IDX4(b, n, y, xx, C_a, H, W)] = m;
                }
}

/* Backward pass of the forward above (one-layer estimator, depth-wise LK; Eq. 4), by the chain rule written
 * out.  With go = dL/dout [B,C,H,W], Wm[b,c] = LK[c] + ZP(dk[b,c]) and x~ the zero-padded input:
 *   g_tap[b,c,i,j] = sum_{y,x} go[b,c,y,x] * x~[b,c,y+i-P,x+j-P]              (per-image tap gradient)
 *   g_lk[c,i,j]    = sum_b g_tap[b,c,i,j]                                      (dL/dLK)
 *   g_dk[b,c,i,j]  = g_tap[b,c,i+P-1,j+P-1]                                    (its central 3x3: dL/ddk)
 *   g_b[o]         = sum_b g_dk[b,o]            g_W[o,k] = sum_b g_dk[b,o] * g[b,k]
 *   g_g[b,k]       = sum_o W[o,k] * g_dk[b,o]
 *   g_x[b,c,y,x]   = sum_{i,j} Wm[b,c,i,j] * go~[b,c,y-(i-P),x-(j-P)] + g_g[b,c] / (H*W)      c < C_a
 *   g_x[b,c]       = go[b,c]                                                                   c >= C_a
 * Outputs: gx [B,C,H,W], glk [C_a,K,K], gw [9*C_a,C_a], gb [9*C_a]; any of them may be NULL. */
void convattn_ref_backward(const float *x, const float *go, int B, int C, int C_a, int H, int W, int K,
                           const double *w_large, const double *w_dyn, const double *b_dyn,
                           double *gx, double *glk, double *gw, double *gb)
{
    const int P = (K - 1) / 2;
    const size_t nt = (size_t)B * C_a * K * K;
    double *g = (double *)malloc(sizeof(double) * (size_t)B * C_a);
    double *dk = (double *)malloc(sizeof(double) * (size_t)B * C_a * 9);
    double *gtap = (double *)malloc(sizeof(double) * nt);
    double *gg = (double *)malloc(sizeof(double) * (size_t)B * C_a);
    convattn_ref_gap(x, B, C, C_a, H, W, g);
    convattn_ref_dynkernel(g, B, C_a, w_dyn, b_dyn, dk);
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C_a; ++c)
            for (int i = 0; i < K; ++i)
                for (int j = 0; j < K; ++j) {
                    double s = 0.0;
                    for (int y = 0; y < H; ++y)
                        for (int xx = 0; xx < W; ++xx) {
                            int yy = y + i - P, xc = xx + j - P;
                            if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                s += (double)go[IDX4(b, c, y, xx, C, H, W)] * (double)x[IDX4(b, c, yy, xc, C, H, W)];
                        }
                    gtap[(((size_t)b * C_a + c) * K + i) * K + j] = s;
                }
    if (glk)
        for (int c = 0; c < C_a; ++c)
            for (int t = 0; t < K * K; ++t) {
                double s = 0.0;
                for (int b = 0; b < B; ++b) s += gtap[((size_t)b * C_a + c) * K * K + t];
                glk[(size_t)c * K * K + t] = s;
            }
    /* dL/ddk[b,o], o = c*9 + i*3 + j: the central 3x3 of the tap gradient (zero where K < 3 leaves no such tap) */
#define GDK(b, c, i, j) (((i) + P - 1 >= 0 && (i) + P - 1 < K && (j) + P - 1 >= 0 && (j) + P - 1 < K) \
                             ? gtap[(((size_t)(b) * C_a + (c)) * K + (i) + P - 1) * K + (j) + P - 1] : 0.0)
    /* for K = 1 the dynamic taps other than the centre have no LK counterpart: take them directly */
    double *gdk = (double *)malloc(sizeof(double) * (size_t)B * C_a * 9);
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C_a; ++c)
            for (int i = 0; i < 3; ++i)
                for (int j = 0; j < 3; ++j) {
                    double s;
                    if (K >= 3) s = GDK(b, c, i, j);
                    else {
                        s = 0.0;
                        for (int y = 0; y < H; ++y)
                            for (int xx = 0; xx < W; ++xx) {
                                int yy = y + i - 1, xc = xx + j - 1;
                                if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                    s += (double)go[IDX4(b, c, y, xx, C, H, W)] * (double)x[IDX4(b, c, yy, xc, C, H, W)];
                            }
                    }
                    gdk[((size_t)b * C_a + c) * 9 + i * 3 + j] = s;
                }
#undef GDK
    if (gb)
        for (int o = 0; o < 9 * C_a; ++o) {
            double s = 0.0;
            for (int b = 0; b < B; ++b) s += gdk[(size_t)b * 9 * C_a + o];
            gb[o] = s;
        }
    if (gw)
        for (int o = 0; o < 9 * C_a; ++o)
            for (int k = 0; k < C_a; ++k) {
                double s = 0.0;
                for (int b = 0; b < B; ++b) s += gdk[(size_t)b * 9 * C_a + o] * g[(size_t)b * C_a + k];
                gw[(size_t)o * C_a + k] = s;
            }
    for (int b = 0; b < B; ++b)
        for (int k = 0; k < C_a; ++k) {
            double s = 0.0;
            for (int o = 0; o < 9 * C_a; ++o) s += w_dyn[(size_t)o * C_a + k] * gdk[(size_t)b * 9 * C_a + o];
            gg[(size_t)b * C_a + k] = s;
        }
    if (gx) {
#pragma omp parallel for collapse(3) schedule(static)
        for (int b = 0; b < B; ++b)
            for (int c = 0; c < C; ++c)
                for (int y = 0; y < H; ++y)
                    for (int xx = 0; xx < W; ++xx) {
                        if (c >= C_a) {
                            gx[IDX4(b, c, y, xx, C, H, W)] = (double)go[IDX4(b, c, y, xx, C, H, W)];
                            continue;
                        }
                        double s = 0.0;
                        for (int i = 0; i < K; ++i)
                            for (int j = 0; j < K; ++j) {
                                int yy = y - (i - P), xc = xx - (j - P);
                                if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                    s += w_large[((size_t)c * K + i) * K + j] * (double)go[IDX4(b, c, yy, xc, C, H, W)];
                            }
                        for (int i = 0; i < 3; ++i)
                            for (int j = 0; j < 3; ++j) {
                                int yy = y - (i - 1), xc = xx - (j - 1);
                                if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                    s += dk[((size_t)b * C_a + c) * 9 + i * 3 + j] * (double)go[IDX4(b, c, yy, xc, C, H, W)];
                            }
                        gx[IDX4(b, c, y, xx, C, H, W)] = s + gg[(size_t)b * C_a + c] / ((double)H * (double)W);
                    }
    }
    free(g); free(dk); free(gtap); free(gg); free(gdk);
}

/* Derivative of the Gaussian error linear unit phi(t) = t * Phi(t): phi'(t) = Phi(t) + t * n(t), n the standard
 * normal density. */
static double gelu_prime(double t)
{
    return 0.5 * erfc(-t / sqrt(2.0)) + t * exp(-0.5 * t * t) / sqrt(2.0 * 3.14159265358979323846);
}

/* Backward pass of the forward with the estimator as Eq. 4 line 2 writes it (two layers, GELU between them; depth-wise
 * LK), by the chain rule written out.  With g = GAP(x), t = W_down g + b_down, a = phi(t), dk = W_up a + b_up, and
 * g_tap, g_lk, g_dk as in convattn_ref_backward:
 *   g_bu[o]   = sum_b g_dk[b,o]                   g_Wu[o,m] = sum_b g_dk[b,o] * a[b,m]
 *   g_a[b,m]  = sum_o W_up[o,m] * g_dk[b,o]       g_t[b,m]  = g_a[b,m] * phi'(t[b,m])
 *   g_bd[m]   = sum_b g_t[b,m]                    g_Wd[m,k] = sum_b g_t[b,m] * g[b,k]
 *   g_g[b,k]  = sum_m W_down[m,k] * g_t[b,m]
 *   g_x[b,c,y,x] = sum_{i,j} Wm[b,c,i,j] * go~[b,c,y-(i-P),x-(j-P)] + g_g[b,c] / (H*W)   (c < C_a);   g_x[b,c] = go[b,c]  (c >= C_a)
 * Outputs: gx [B,C,H,W], glk [C_a,K,K], gwd [h,C_a], gbd [h], gwu [9*C_a,h], gbu [9*C_a]; any may be NULL.  K >= 3. */
void convattn_ref_backward_mlp(const float *x, const float *go, int B, int C, int C_a, int H, int W, int K,
                               const double *w_large, int h, const double *w_down, const double *b_down,
                               const double *w_up, const double *b_up,
                               double *gx, double *glk, double *gwd, double *gbd, double *gwu, double *gbu)
{
    const int P = (K - 1) / 2;
    double *g = (double *)malloc(sizeof(double) * (size_t)B * C_a);
    double *t = (double *)malloc(sizeof(double) * (size_t)B * h);
    double *a = (double *)malloc(sizeof(double) * (size_t)B * h);
    double *dk = (double *)malloc(sizeof(double) * (size_t)B * C_a * 9);
    double *gtap = (double *)malloc(sizeof(double) * (size_t)B * C_a * K * K);
    double *gdk = (double *)malloc(sizeof(double) * (size_t)B * C_a * 9);
    double *gt = (double *)malloc(sizeof(double) * (size_t)B * h);
    double *gg = (double *)malloc(sizeof(double) * (size_t)B * C_a);
    /* forward quantities */
    convattn_ref_gap(x, B, C, C_a, H, W, g);
    for (int b = 0; b < B; ++b) {
        for (int m = 0; m < h; ++m) {
            double s = b_down[m];
            for (int k = 0; k < C_a; ++k) s += w_down[(size_t)m * C_a + k] * g[(size_t)b * C_a + k];
            t[(size_t)b * h + m] = s;
            a[(size_t)b * h + m] = gelu(s);
        }
        for (int o = 0; o < 9 * C_a; ++o) {
            double s = b_up[o];
            for (int m = 0; m < h; ++m) s += w_up[(size_t)o * h + m] * a[(size_t)b * h + m];
            dk[(size_t)b * 9 * C_a + o] = s;
        }
    }
    /* per-image tap gradients */
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C_a; ++c)
            for (int i = 0; i < K; ++i)
                for (int j = 0; j < K; ++j) {
                    double s = 0.0;
                    for (int y = 0; y < H; ++y)
                        for (int xx = 0; xx < W; ++xx) {
                            int yy = y + i - P, xc = xx + j - P;
                            if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                s += (double)go[IDX4(b, c, y, xx, C, H, W)] * (double)x[IDX4(b, c, yy, xc, C, H, W)];
                        }
                    gtap[(((size_t)b * C_a + c) * K + i) * K + j] = s;
                }
    if (glk)
        for (int c = 0; c < C_a; ++c)
            for (int q = 0; q < K * K; ++q) {
                double s = 0.0;
                for (int b = 0; b < B; ++b) s += gtap[((size_t)b * C_a + c) * K * K + q];
                glk[(size_t)c * K * K + q] = s;
            }
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C_a; ++c)
            for (int i = 0; i < 3; ++i)
                for (int j = 0; j < 3; ++j)
                    gdk[((size_t)b * C_a + c) * 9 + i * 3 + j] = gtap[(((size_t)b * C_a + c) * K + i + P - 1) * K + j + P - 1];
    /* second layer */
    if (gbu)
        for (int o = 0; o < 9 * C_a; ++o) {
            double s = 0.0;
            for (int b = 0; b < B; ++b) s += gdk[(size_t)b * 9 * C_a + o];
            gbu[o] = s;
        }
    if (gwu)
        for (int o = 0; o < 9 * C_a; ++o)
            for (int m = 0; m < h; ++m) {
                double s = 0.0;
                for (int b = 0; b < B; ++b) s += gdk[(size_t)b * 9 * C_a + o] * a[(size_t)b * h + m];
                gwu[(size_t)o * h + m] = s;
            }
    /* through the activation */
    for (int b = 0; b < B; ++b)
        for (int m = 0; m < h; ++m) {
            double s = 0.0;
            for (int o = 0; o < 9 * C_a; ++o) s += w_up[(size_t)o * h + m] * gdk[(size_t)b * 9 * C_a + o];
            gt[(size_t)b * h + m] = s * gelu_prime(t[(size_t)b * h + m]);
        }
    /* first layer */
    if (gbd)
        for (int m = 0; m < h; ++m) {
            double s = 0.0;
            for (int b = 0; b < B; ++b) s += gt[(size_t)b * h + m];
            gbd[m] = s;
        }
    if (gwd)
        for (int m = 0; m < h; ++m)
            for (int k = 0; k < C_a; ++k) {
                double s = 0.0;
                for (int b = 0; b < B; ++b) s += gt[(size_t)b * h + m] * g[(size_t)b * C_a + k];
                gwd[(size_t)m * C_a + k] = s;
            }
    for (int b = 0; b < B; ++b)
        for (int k = 0; k < C_a; ++k) {
            double s = 0.0;
            for (int m = 0; m < h; ++m) s += w_down[(size_t)m * C_a + k] * gt[(size_t)b * h + m];
            gg[(size_t)b * C_a + k] = s;
        }
    if (gx) {
#pragma omp parallel for collapse(3) schedule(static)
        for (int b = 0; b < B; ++b)
            for (int c = 0; c < C; ++c)
                for (int y = 0; y < H; ++y)
                    for (int xx = 0; xx < W; ++xx) {
                        if (c >= C_a) {
                            gx[IDX4(b, c, y, xx, C, H, W)] = (double)go[IDX4(b, c, y, xx, C, H, W)];
                            continue;
                        }
                        double s = 0.0;
                        for (int i = 0; i < K; ++i)
                            for (int j = 0; j < K; ++j) {
                                int yy = y - (i - P), xc = xx - (j - P);
                                if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                    s += w_large[((size_t)c * K + i) * K + j] * (double)go[IDX4(b, c, yy, xc, C, H, W)];
                            }
                        for (int i = 0; i < 3; ++i)
                            for (int j = 0; j < 3; ++j) {
                                int yy = y - (i - 1), xc = xx - (j - 1);
                                if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                    s += dk[((size_t)b * C_a + c) * 9 + i * 3 + j] * (double)go[IDX4(b, c, yy, xc, C, H, W)];
                            }
                        gx[IDX4(b, c, y, xx, C, H, W)] = s + gg[(size_t)b * C_a + c] / ((double)H * (double)W);
                    }
    }
    free(g); free(t); free(a); free(dk); free(gtap); free(gdk); free(gt); free(gg);
}

/* Backward pass of the decomposed form of Eq. 5 (point-wise LK^c in front of the depth-wise stage, one-layer
 * estimator), by the chain rule written out.  With m[b,n] = sum_k w_point[n,k] * x[b,k] (the mixed features, exact),
 * g = GAP(x) of the UNMIXED features, dk = W g + b, Wm[b,n] = LK[n] + ZP(dk[b,n]) and m~, go~ zero-padded:
 *   g_tap[b,n,i,j] = sum_{y,x} go[b,n,y,x] * m~[b,n,y+i-P,x+j-P]
 *   g_lk[n,i,j]    = sum_b g_tap[b,n,i,j]         g_dk[b,n,i,j] = g_tap[b,n,i+P-1,j+P-1]
 *   g_b[o]         = sum_b g_dk[b,o]              g_W[o,k]      = sum_b g_dk[b,o] * g[b,k]
 *   g_g[b,k]       = sum_o W[o,k] * g_dk[b,o]
 *   g_m[b,n,y,x]   = sum_{i,j} Wm[b,n,i,j] * go~[b,n,y-(i-P),x-(j-P)]         (dL/dm)
 *   g_P[n,k]       = sum_{b,y,x} g_m[b,n,y,x] * x[b,k,y,x]                    (dL/dLK^c)
 *   g_x[b,k,y,x]   = sum_n w_point[n,k] * g_m[b,n,y,x] + g_g[b,k] / (H*W)     k < C_a
 *   g_x[b,c]       = go[b,c]                                                  c >= C_a
 * Outputs: gx [B,C,H,W], glk [C_a,K,K], gwp [C_a,C_a], gw [9*C_a,C_a], gb [9*C_a]; any may be NULL.  K >= 3. */
void convattn_ref_backward_pw(const float *x, const float *go, int B, int C, int C_a, int H, int W, int K,
                              const double *w_large, const double *w_point, const double *w_dyn, const double *b_dyn,
                              double *gx, double *glk, double *gwp, double *gw, double *gb)
{
    const int P = (K - 1) / 2;
    const size_t HW = (size_t)H * W;
    double *g = (double *)malloc(sizeof(double) * (size_t)B * C_a);
    double *dk = (double *)malloc(sizeof(double) * (size_t)B * C_a * 9);
    double *m = (double *)malloc(sizeof(double) * (size_t)B * C_a * HW);
    double *gm = (double *)malloc(sizeof(double) * (size_t)B * C_a * HW);
    double *gtap = (double *)malloc(sizeof(double) * (size_t)B * C_a * K * K);
    double *gdk = (double *)malloc(sizeof(double) * (size_t)B * C_a * 9);
    double *gg = (double *)malloc(sizeof(double) * (size_t)B * C_a);
    convattn_ref_gap(x, B, C, C_a, H, W, g);
    convattn_ref_dynkernel(g, B, C_a, w_dyn, b_dyn, dk);
    /* the mixed features */
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < C_a; ++n)
            for (size_t q = 0; q < HW; ++q) {
                double s = 0.0;
                for (int k = 0; k < C_a; ++k)
                    s += w_point[(size_t)n * C_a + k] * (double)x[((size_t)b * C + k) * HW + q];
                m[((size_t)b * C_a + n) * HW + q] = s;
            }
    /* tap gradients against the mixed features */
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < C_a; ++n)
            for (int i = 0; i < K; ++i)
                for (int j = 0; j < K; ++j) {
                    double s = 0.0;
                    for (int y = 0; y < H; ++y)
                        for (int xx = 0; xx < W; ++xx) {
                            int yy = y + i - P, xc = xx + j - P;
                            if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                s += (double)go[IDX4(b, n, y, xx, C, H, W)] * m[((size_t)b * C_a + n) * HW + (size_t)yy * W + xc];
                        }
                    gtap[(((size_t)b * C_a + n) * K + i) * K + j] = s;
                }
    if (glk)
        for (int n = 0; n < C_a; ++n)
            for (int t = 0; t < K * K; ++t) {
                double s = 0.0;
                for (int b = 0; b < B; ++b) s += gtap[((size_t)b * C_a + n) * K * K + t];
                glk[(size_t)n * K * K + t] = s;
            }
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < C_a; ++n)
            for (int i = 0; i < 3; ++i)
                for (int j = 0; j < 3; ++j)
                    gdk[((size_t)b * C_a + n) * 9 + i * 3 + j] = gtap[(((size_t)b * C_a + n) * K + i + P - 1) * K + j + P - 1];
    if (gb)
        for (int o = 0; o < 9 * C_a; ++o) {
            double s = 0.0;
            for (int b = 0; b < B; ++b) s += gdk[(size_t)b * 9 * C_a + o];
            gb[o] = s;
        }
    if (gw)
        for (int o = 0; o < 9 * C_a; ++o)
            for (int k = 0; k < C_a; ++k) {
                double s = 0.0;
                for (int b = 0; b < B; ++b) s += gdk[(size_t)b * 9 * C_a + o] * g[(size_t)b * C_a + k];
                gw[(size_t)o * C_a + k] = s;
            }
    for (int b = 0; b < B; ++b)
        for (int k = 0; k < C_a; ++k) {
            double s = 0.0;
            for (int o = 0; o < 9 * C_a; ++o) s += w_dyn[(size_t)o * C_a + k] * gdk[(size_t)b * 9 * C_a + o];
            gg[(size_t)b * C_a + k] = s;
        }
    /* dL/dm: the depth-wise stage's adjoint */
#pragma omp parallel for collapse(3) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < C_a; ++n)
            for (int y = 0; y < H; ++y)
                for (int xx = 0; xx < W; ++xx) {
                    double s = 0.0;
                    for (int i = 0; i < K; ++i)
                        for (int j = 0; j < K; ++j) {
                            int yy = y - (i - P), xc = xx - (j - P);
                            if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                s += w_large[((size_t)n * K + i) * K + j] * (double)go[IDX4(b, n, yy, xc, C, H, W)];
                        }
                    for (int i = 0; i < 3; ++i)
                        for (int j = 0; j < 3; ++j) {
                            int yy = y - (i - 1), xc = xx - (j - 1);
                            if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                s += dk[((size_t)b * C_a + n) * 9 + i * 3 + j] * (double)go[IDX4(b, n, yy, xc, C, H, W)];
                        }
                    gm[((size_t)b * C_a + n) * HW + (size_t)y * W + xx] = s;
                }
    if (gwp)
        for (int n = 0; n < C_a; ++n)
            for (int k = 0; k < C_a; ++k) {
                double s = 0.0;
                for (int b = 0; b < B; ++b)
                    for (size_t q = 0; q < HW; ++q)
                        s += gm[((size_t)b * C_a + n) * HW + q] * (double)x[((size_t)b * C + k) * HW + q];
                gwp[(size_t)n * C_a + k] = s;
            }
    if (gx) {
#pragma omp parallel for collapse(2) schedule(static)
        for (int b = 0; b < B; ++b)
            for (int c = 0; c < C; ++c)
                for (size_t q = 0; q < HW; ++q) {
                    if (c >= C_a) {
                        gx[((size_t)b * C + c) * HW + q] = (double)go[((size_t)b * C + c) * HW + q];
                        continue;
                    }
                    double s = 0.0;
                    for (int n = 0; n < C_a; ++n)
                        s += w_point[(size_t)n * C_a + c] * gm[((size_t)b * C_a + n) * HW + q];
                    gx[((size_t)b * C + c) * HW + q] = s + gg[(size_t)b * C_a + c] / ((double)H * (double)W);
                }
    }
    free(g); free(dk); free(m); free(gm); free(gtap); free(gdk); free(gg);
}

/* Backward pass of the forward with the dense large kernel of Section 3.2 (w_dense[n,k,i,j]: output channel n sums
 * over every attention input channel k; the dynamic 3x3 kernel stays depth-wise; one-layer estimator), by the chain rule
 * written out.  With go = dL/dout, x~ and go~ zero-padded, g = GAP(x), dk = W g + b:
 *   g_wd[n,k,i,j] = sum_{b,y,x} go[b,n,y,x] * x~[b,k,y+i-P,x+j-P]                         (dL/dw_dense)
 *   g_dk[b,c,i,j] = sum_{y,x} go[b,c,y,x] * x~[b,c,y+i-1,x+j-1]                           (dL/ddk, depth-wise)
 *   g_b[o] = sum_b g_dk[b,o]     g_W[o,k] = sum_b g_dk[b,o] * g[b,k]     g_g[b,k] = sum_o W[o,k] * g_dk[b,o]
 *   g_x[b,k,y,x]  = sum_n sum_{i,j} w_dense[n,k,i,j] * go~[b,n,y-(i-P),x-(j-P)]
 *                 + sum_{i,j} dk[b,k,i,j] * go~[b,k,y-(i-1),x-(j-1)] + g_g[b,k] / (H*W)     k < C_a
 *   g_x[b,c]      = go[b,c]                                                                c >= C_a
 * Outputs: gx [B,C,H,W], gwd [C_a,C_a,K,K], gw [9*C_a,C_a], gb [9*C_a]; any may be NULL. */
void convattn_ref_backward_dense(const float *x, const float *go, int B, int C, int C_a, int H, int W, int K,
                                 const double *w_dense, const double *w_dyn, const double *b_dyn,
                                 double *gx, double *gwd, double *gw, double *gb)
{
    const int P = (K - 1) / 2;
    double *g = (double *)malloc(sizeof(double) * (size_t)B * C_a);
    double *dk = (double *)malloc(sizeof(double) * (size_t)B * C_a * 9);
    double *gdk = (double *)malloc(sizeof(double) * (size_t)B * C_a * 9);
    double *gg = (double *)malloc(sizeof(double) * (size_t)B * C_a);
    convattn_ref_gap(x, B, C, C_a, H, W, g);
    convattn_ref_dynkernel(g, B, C_a, w_dyn, b_dyn, dk);
    if (gwd) {
#pragma omp parallel for collapse(2) schedule(static)
        for (int n = 0; n < C_a; ++n)
            for (int k = 0; k < C_a; ++k)
                for (int i = 0; i < K; ++i)
                    for (int j = 0; j < K; ++j) {
                        double s = 0.0;
                        for (int b = 0; b < B; ++b)
                            for (int y = 0; y < H; ++y)
                                for (int xx = 0; xx < W; ++xx) {
                                    int yy = y + i - P, xc = xx + j - P;
                                    if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                        s += (double)go[IDX4(b, n, y, xx, C, H, W)] * (double)x[IDX4(b, k, yy, xc, C, H, W)];
                                }
                        gwd[(((size_t)n * C_a + k) * K + i) * K + j] = s;
                    }
    }
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C_a; ++c)
            for (int i = 0; i < 3; ++i)
                for (int j = 0; j < 3; ++j) {
                    double s = 0.0;
                    for (int y = 0; y < H; ++y)
                        for (int xx = 0; xx < W; ++xx) {
                            int yy = y + i - 1, xc = xx + j - 1;
                            if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                s += (double)go[IDX4(b, c, y, xx, C, H, W)] * (double)x[IDX4(b, c, yy, xc, C, H, W)];
                        }
                    gdk[((size_t)b * C_a + c) * 9 + i * 3 + j] = s;
                }
    if (gb)
        for (int o = 0; o < 9 * C_a; ++o) {
            double s = 0.0;
            for (int b = 0; b < B; ++b) s += gdk[(size_t)b * 9 * C_a + o];
            gb[o] = s;
        }
    if (gw)
        for (int o = 0; o < 9 * C_a; ++o)
            for (int k = 0; k < C_a; ++k) {
                double s = 0.0;
                for (int b = 0; b < B; ++b) s += gdk[(size_t)b * 9 * C_a + o] * g[(size_t)b * C_a + k];
                gw[(size_t)o * C_a + k] = s;
            }
    for (int b = 0; b < B; ++b)
        for (int k = 0; k < C_a; ++k) {
            double s = 0.0;
            for (int o = 0; o < 9 * C_a; ++o) s += w_dyn[(size_t)o * C_a + k] * gdk[(size_t)b * 9 * C_a + o];
            gg[(size_t)b * C_a + k] = s;
        }
    if (gx) {
#pragma omp parallel for collapse(3) schedule(static)
        for (int b = 0; b < B; ++b)
            for (int c = 0; c < C; ++c)
                for (int y = 0; y < H; ++y)
                    for (int xx = 0; xx < W; ++xx) {
                        if (c >= C_a) {
                            gx[IDX4(b, c, y, xx, C, H, W)] = (double)go[IDX4(b, c, y, xx, C, H, W)];
                            continue;
                        }
                        double s = 0.0;
                        for (int n = 0; n < C_a; ++n)
                            for (int i = 0; i < K; ++i)
                                for (int j = 0; j < K; ++j) {
                                    int yy = y - (i - P), xc = xx - (j - P);
                                    if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                        s += w_dense[(((size_t)n * C_a + c) * K + i) * K + j] * (double)go[IDX4(b, n, yy, xc, C, H, W)];
                                }
                        for (int i = 0; i < 3; ++i)
                            for (int j = 0; j < 3; ++j) {
                                int yy = y - (i - 1), xc = xx - (j - 1);
                                if (yy >= 0 && yy < H && xc >= 0 && xc < W)
                                    s += dk[((size_t)b * C_a + c) * 9 + i * 3 + j] * (double)go[IDX4(b, c, yy, xc, C, H, W)];
                            }
                        gx[IDX4(b, c, y, xx, C, H, W)] = s + gg[(size_t)b * C_a + c] / ((double)H * (double)W);
                    }
    }
    free(g); free(dk); free(gdk); free(gg);
}

/* Selected entries of the dense kernel's gradient, one by one (for sizes where the whole of convattn_ref_backward_dense
 * takes too long): idx[t] is a flat index into g_wd[C_a,C_a,K,K];
 *   vals[t] = sum_{b,y,x} go[b,n,y,x] * x~[b,k,y+i-P,x+j-P],   mags[t] (optional) the same sum of magnitudes. */
void convattn_ref_backward_dense_points(const float *x, const float *go, int B, int C, int C_a, int H, int W, int K,
                                        int64_t n_idx, const int64_t *idx, double *vals, double *mags)
{
    const int P = (K - 1) / 2;
#pragma omp parallel for schedule(dynamic)
    for (int64_t t = 0; t < n_idx; ++t) {
        int64_t f = idx[t];
        int j = (int)(f % K); f /= K;
        int i = (int)(f % K); f /= K;
        int k = (int)(f % C_a); f /= C_a;
        int n = (int)f;
        double s = 0.0, m = 0.0;
        for (int b = 0; b < B; ++b)
            for (int y = 0; y < H; ++y)
                for (int xx = 0; xx < W; ++xx) {
                    int yy = y + i - P, xc = xx + j - P;
                    if (yy >= 0 && yy < H && xc >= 0 && xc < W) {
                        double v = (double)go[IDX4(b, n, y, xx, C, H, W)] * (double)x[IDX4(b, k, yy, xc, C, H, W)];
                        s += v;
                        m += fabs(v);
                    }
                }
        vals[t] = s;
        if (mags) mags[t] = m;
    }
}

/* Selected outputs, one by one: idx[n] are flat indices into out[B,C,H,W]; dk is
 * given (from convattn_ref_gap + convattn_ref_dynkernel). */
void convattn_ref_points(const float *x, int B, int C, int C_a, int H, int W, int K,
                         const double *w_large, const double *dk, int64_t n, const int64_t *idx,
                         double *vals, double *mags)
{
    (void)B;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n; ++t) {
        int64_t f = idx[t];
        int xx = (int)(f % W); f /= W;
        int y = (int)(f % H);  f /= H;
        int c = (int)(f % C);  f /= C;
        int b = (int)f;
        double m = 0.0;
        if (c < C_a)
            vals[t] = one_output(x, C, H, W, K, w_large, dk + (size_t)b * 9 * C_a, b, c, y, xx, &m);
        else {
            vals[t] = (double)x[IDX4(b, c, y, xx, C, H, W)];
            m = fabs(vals[t]);
        }
        if (mags) mags[t] = m;
    }
}

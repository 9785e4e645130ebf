/*
 * CPU oracle for the key-frame partial-distillation step of ShadowTutor.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct
 * statement of what the CUDA path has to compute.  It shares no code with the
 * CUDA library and is never on the product path: only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may load it.
 *
 * What it states (paper passages):
 *   - pseudo-label = teacher output reduced to one class per pixel
 *     (Section 4.1.2 "Teacher inference", Algorithm 3 "label <- Forward(teacher)");
 *     one byte per pixel (Table 4, 0.879 MB for a 1280x720 label map);
 *   - one iteration of Algorithm 1's loop body: Forward, ComputeLoss (per-pixel
 *     cross-entropy, Section 5.2), PartialBackward (gradients only for the
 *     non-frozen back part, Section 4.2), OptimStep (gradient descent,
 *     Section 4.1.4), ComputeMetric (mean IoU, Section 3.2 equation for IoU_c);
 *   - UpdatedPart(student): the trained subset as fp32 values (Algorithm 3, Table 4).
 *
 * Storage type `real` is float (default) or double (-DST_REAL=double); every long
 * sum (convolution dot products, loss, weight/bias gradients) is accumulated in
 * double.  Compile with -ffp-contract=off so no multiply-add is fused.
 * Loops are written in the order of the definitions; OpenMP only splits
 * independent outputs.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef ST_REAL
#define ST_REAL float
#endif
typedef ST_REAL real;

int so_sizeof_real(void) { return (int)sizeof(real); }

/* ---------------------------------------------------------------------------
 * Pseudo-label: label[p] = argmax_c T[c][p], lowest class index on ties
 * (Algorithm 3: label <- Forward(teacher, frame); Table 4: 1 byte per pixel).
 * T is [C][P] planar, P = H*W.
 * ------------------------------------------------------------------------- */
void so_labels(const real *T, int C, int64_t P, uint8_t *out)
{
#pragma omp parallel for
    for (int64_t p = 0; p < P; ++p) {
        real best = T[p];
        int idx = 0;
        for (int c = 1; c < C; ++c) {
            real v = T[(int64_t)c * P + p];
            if (v > best) { best = v; idx = c; }
        }
        out[p] = (uint8_t)idx;
    }
}

/* ---------------------------------------------------------------------------
 * Head convolution (Forward of the trainable back part, Algorithm 1):
 *   out[co][y][x] = b[co] + sum_{ci,ky,kx} Wt[co][ci][ky][kx] * in[ci][y+ky-r][x+kx-r]
 * with zero padding r = ks/2, ks in {1,3}; optional ReLU(v) = max(v, 0).
 * Planar NCHW, weights [Cout][Cin][ks][ks].  One double accumulator per output.
 * ------------------------------------------------------------------------- */
void so_conv_fwd(const real *in, int Cin, int h, int w, const real *Wt, const real *b,
                 int Cout, int ks, int relu, real *out)
{
    const int r = ks / 2;
#pragma omp parallel for
    for (int co = 0; co < Cout; ++co) {
        double *acc = (double *)malloc(sizeof(double) * (size_t)w);
        for (int y = 0; y < h; ++y) {
            for (int x = 0; x < w; ++x) acc[x] = 0.0;
            for (int ci = 0; ci < Cin; ++ci)
                for (int ky = 0; ky < ks; ++ky) {
                    int yy = y + ky - r;
                    if (yy < 0 || yy >= h) continue;          /* zero padding */
                    for (int kx = 0; kx < ks; ++kx) {
                        double wv = (double)Wt[(((int64_t)co * Cin + ci) * ks + ky) * ks + kx];
                        const real *row = in + ((int64_t)ci * h + yy) * w;
                        for (int x = 0; x < w; ++x) {
                            int xx = x + kx - r;
                            if (xx < 0 || xx >= w) continue;  /* zero padding */
                            acc[x] += wv * (double)row[xx];
                        }
                    }
                }
            for (int x = 0; x < w; ++x) {
                real v = (real)(acc[x] + (double)b[co]);
                if (relu && !(v > (real)0)) v = (real)0;
                out[((int64_t)co * h + y) * w + x] = v;
            }
        }
        free(acc);
    }
}

/* ---------------------------------------------------------------------------
 * Bilinear upsample by an integer factor s, half-pixel centres
 * ("align_corners = false"): for output index Y
 *   src = (Y + 0.5)/s - 0.5, clamped below at 0; y0 = floor(src);
 *   y1 = y0 + (y0 < h-1); lambda = src - y0,
 * same along x; horizontal interpolation first, then vertical.
 * The head's low-resolution logits are brought to frame resolution this way
 * before the per-pixel loss (prediction has the frame's spatial size, Section 3.2).
 * ------------------------------------------------------------------------- */
static void src_index(int64_t Y, int s, int n, int *i0, int *i1, real *lam)
{
    real src = ((real)Y + (real)0.5) / (real)s - (real)0.5;
    if (src < (real)0) src = (real)0;
    int a = (int)floor((double)src);
    if (a > n - 1) a = n - 1;
    *i0 = a;
    *i1 = a + (a < n - 1 ? 1 : 0);
    *lam = src - (real)a;
}

void so_upsample(const real *z, int C, int h, int w, int s, real *u)
{
    const int H = h * s, W = w * s;
#pragma omp parallel for
    for (int c = 0; c < C; ++c)
        for (int Y = 0; Y < H; ++Y) {
            int y0, y1; real ly;
            src_index(Y, s, h, &y0, &y1, &ly);
            for (int X = 0; X < W; ++X) {
                int x0, x1; real lx;
                src_index(X, s, w, &x0, &x1, &lx);
                const real *zc = z + (int64_t)c * h * w;
                real top = ((real)1 - lx) * zc[(int64_t)y0 * w + x0] + lx * zc[(int64_t)y0 * w + x1];
                real bot = ((real)1 - lx) * zc[(int64_t)y1 * w + x0] + lx * zc[(int64_t)y1 * w + x1];
                u[((int64_t)c * H + Y) * W + X] = ((real)1 - ly) * top + ly * bot;
            }
        }
}

/* Exact transpose of so_upsample: dz = U^T g (scatter with the same four weights). */
void so_upsample_adjoint(const real *g, int C, int h, int w, int s, real *dz)
{
    const int H = h * s, W = w * s;
#pragma omp parallel for
    for (int c = 0; c < C; ++c) {
        double *acc = (double *)calloc((size_t)h * w, sizeof(double));
        for (int Y = 0; Y < H; ++Y) {
            int y0, y1; real ly;
            src_index(Y, s, h, &y0, &y1, &ly);
            for (int X = 0; X < W; ++X) {
                int x0, x1; real lx;
                src_index(X, s, w, &x0, &x1, &lx);
                double gv = (double)g[((int64_t)c * H + Y) * W + X];
                double wy0 = 1.0 - (double)ly, wy1 = (double)ly;
                double wx0 = 1.0 - (double)lx, wx1 = (double)lx;
                acc[(int64_t)y0 * w + x0] += wy0 * wx0 * gv;
                acc[(int64_t)y0 * w + x1] += wy0 * wx1 * gv;
                acc[(int64_t)y1 * w + x0] += wy1 * wx0 * gv;
                acc[(int64_t)y1 * w + x1] += wy1 * wx1 * gv;
            }
        }
        for (int64_t i = 0; i < (int64_t)h * w; ++i) dz[(int64_t)c * h * w + i] = (real)acc[i];
        free(acc);
    }
}

/* ---------------------------------------------------------------------------
 * ComputeLoss (Algorithm 1; Section 5.2: cross-entropy against the pseudo-label),
 * unweighted mean over all P pixels, and its gradient w.r.t. the logits:
 *   m = max_c u_c; Z = sum_c exp(u_c - m); loss_p = m + log Z - u_label;
 *   g_c = (exp(u_c - m)/Z - [c == label]) / P.
 * u is [C][P]; g (may be NULL) is [C][P]; *loss = (1/P) sum_p loss_p.
 * Returns the number of labels >= C (those pixels are skipped).
 * ------------------------------------------------------------------------- */
int64_t so_softmax_ce_weighted(const real *u, const uint8_t *lab, const uint8_t *wgt, int C, int64_t P, real *g, double *loss);

int64_t so_softmax_ce(const real *u, const uint8_t *lab, int C, int64_t P, real *g, double *loss)
{
    return so_softmax_ce_weighted(u, lab, NULL, C, P, g, loss);
}

/* ---------------------------------------------------------------------------
 * Loss weighting against class imbalance (Section 5.2): the cross-entropy of pixels "near and within
 * non-background objects" is scaled by a factor (5 in the paper).  wgt[p] is that factor per pixel
 * (NULL: 1 everywhere); the loss of a pixel and its gradient are both multiplied by it, the normaliser stays P:
 *   loss = (1/P) sum_p wgt_p loss_p,   g_c = wgt_p (softmax_c - [c == label]) / P.
 * ------------------------------------------------------------------------- */
int64_t so_softmax_ce_weighted(const real *u, const uint8_t *lab, const uint8_t *wgt, int C, int64_t P, real *g, double *loss)
{
    double total = 0.0;
    int64_t bad = 0;
#pragma omp parallel for reduction(+ : total, bad)
    for (int64_t p = 0; p < P; ++p) {
        int l = lab[p];
        if (l >= C) {
            bad++;
            if (g) for (int c = 0; c < C; ++c) g[(int64_t)c * P + p] = (real)0;
            continue;
        }
        double m = (double)u[p];
        for (int c = 1; c < C; ++c) {
            double v = (double)u[(int64_t)c * P + p];
            if (v > m) m = v;
        }
        double Z = 0.0;
        for (int c = 0; c < C; ++c) Z += exp((double)u[(int64_t)c * P + p] - m);
        const double wp = wgt ? (double)wgt[p] : 1.0;
        total += wp * (m + log(Z) - (double)u[(int64_t)l * P + p]);
        if (g)
            for (int c = 0; c < C; ++c) {
                double pc = exp((double)u[(int64_t)c * P + p] - m) / Z;
                g[(int64_t)c * P + p] = (real)(wp * (pc - (c == l ? 1.0 : 0.0)) / (double)P);
            }
    }
    *loss = total / (double)P;
    return bad;
}

/* ---------------------------------------------------------------------------
 * Which pixels are "near and within non-background objects" (Section 5.2; the paper gives no distance):
 * a pixel gets weight `factor` if any pixel within `radius` rows and columns of it (a square window, cut at the
 * frame border) carries a label other than `background`, weight 1 otherwise.  Brute force over the window.
 * ------------------------------------------------------------------------- */
void so_object_weights(const uint8_t *lab, int H, int W, int background, int radius, int factor, uint8_t *wgt)
{
#pragma omp parallel for
    for (int y = 0; y < H; ++y)
        for (int x = 0; x < W; ++x) {
            int near = 0;
            for (int dy = -radius; dy <= radius && !near; ++dy)
                for (int dx = -radius; dx <= radius; ++dx) {
                    const int yy = y + dy, xx = x + dx;
                    if (yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
                    if (lab[(int64_t)yy * W + xx] != background) { near = 1; break; }
                }
            wgt[(int64_t)y * W + x] = (uint8_t)(near ? factor : 1);
        }
}

/* ---------------------------------------------------------------------------
 * PartialBackward (Algorithm 1; Section 4.2): gradients of the trainable layers only.
 *   dW[co][ci][ky][kx] = sum_{y,x} dout[co][y][x] * in[ci][y+ky-r][x+kx-r]   (zero padding)
 *   db[co]             = sum_{y,x} dout[co][y][x]
 * No gradient is formed for `in` when it is the frozen part's output.
 * ------------------------------------------------------------------------- */
void so_conv_wgrad(const real *in, const real *dout, int Cin, int Cout, int h, int w, int ks,
                   real *dW, real *db)
{
    const int r = ks / 2;
#pragma omp parallel for
    for (int co = 0; co < Cout; ++co) {
        const real *d = dout + (int64_t)co * h * w;
        double sb = 0.0;
        for (int64_t i = 0; i < (int64_t)h * w; ++i) sb += (double)d[i];
        db[co] = (real)sb;
        for (int ci = 0; ci < Cin; ++ci)
            for (int ky = 0; ky < ks; ++ky)
                for (int kx = 0; kx < ks; ++kx) {
                    double acc = 0.0;
                    for (int y = 0; y < h; ++y) {
                        int yy = y + ky - r;
                        if (yy < 0 || yy >= h) continue;
                        const real *row = in + ((int64_t)ci * h + yy) * w;
                        const real *drow = d + (int64_t)y * w;
                        for (int x = 0; x < w; ++x) {
                            int xx = x + kx - r;
                            if (xx < 0 || xx >= w) continue;
                            acc += (double)drow[x] * (double)row[xx];
                        }
                    }
                    dW[(((int64_t)co * Cin + ci) * ks + ky) * ks + kx] = (real)acc;
                }
    }
}

/* db[co] = sum over pixels of dout[co][.] alone (used when dW is formed from rounded operands
 * but the bias gradient from the unrounded ones). */
void so_bias_grad(const real *dout, int Cout, int64_t P, real *db)
{
    for (int co = 0; co < Cout; ++co) {
        double sb = 0.0;
        for (int64_t i = 0; i < P; ++i) sb += (double)dout[(int64_t)co * P + i];
        db[co] = (real)sb;
    }
}

/* Gradient passed from the 1x1 output layer to the hidden activation:
 *   dH[k][p] = sum_c W2[c][k] * dz[c][p];  W2 is [C][Ch], dz [C][P], dH [Ch][P]. */
void so_conv1x1_dgrad(const real *W2, const real *dz, int C, int Ch, int64_t P, real *dH)
{
#pragma omp parallel for
    for (int k = 0; k < Ch; ++k)
        for (int64_t p = 0; p < P; ++p) {
            double acc = 0.0;
            for (int c = 0; c < C; ++c)
                acc += (double)W2[(int64_t)c * Ch + k] * (double)dz[(int64_t)c * P + p];
            dH[(int64_t)k * P + p] = (real)acc;
        }
}

/* Gradient passed back through a convolution layer to its input (needed between trained layers only; nothing is
 * passed back into a frozen layer's output, Section 4.2).  Transpose of so_conv_fwd:
 *   din[ci][y][x] = sum_{co,ky,kx} dout[co][y - ky + r][x - kx + r] * Wt[co][ci][ky][kx]
 * (output pixel (yo, xo) read input pixel (yo + ky - r, xo + kx - r), so input pixel (y, x) was read by output pixel
 * (y - ky + r, x - kx + r); positions outside the map contribute nothing).  Only the first Cin_take input channels
 * are formed (those of the preceding trained layer when the input is a concatenation). */
void so_conv_dgrad(const real *dout, const real *Wt, int Cin, int Cin_take, int Cout, int h, int w, int ks, real *din)
{
    const int r = ks / 2;
#pragma omp parallel for
    for (int ci = 0; ci < Cin_take; ++ci)
        for (int y = 0; y < h; ++y)
            for (int x = 0; x < w; ++x) {
                double acc = 0.0;
                for (int co = 0; co < Cout; ++co)
                    for (int ky = 0; ky < ks; ++ky) {
                        const int yo = y - ky + r;
                        if (yo < 0 || yo >= h) continue;
                        for (int kx = 0; kx < ks; ++kx) {
                            const int xo = x - kx + r;
                            if (xo < 0 || xo >= w) continue;
                            acc += (double)dout[((int64_t)co * h + yo) * w + xo] *
                                   (double)Wt[(((int64_t)co * Cin + ci) * ks + ky) * ks + kx];
                        }
                    }
                din[((int64_t)ci * h + y) * w + x] = (real)acc;
            }
}

/* ReLU backward: the gradient passes where the activation is > 0 (0 at exactly 0). */
void so_relu_mask(real *dH, const real *Hact, int64_t n)
{
    for (int64_t i = 0; i < n; ++i)
        if (!(Hact[i] > (real)0)) dH[i] = (real)0;
}

/* ---------------------------------------------------------------------------
 * OptimStep (Algorithm 1; "most simply gradient descent", Section 4.1.4), with the
 * usual heavy-ball momentum: v <- mu*v + g; theta <- theta - lr*v  (mu = 0: plain SGD).
 * ------------------------------------------------------------------------- */
void so_sgd(real *theta, real *v, const real *g, int64_t n, real lr, real mu)
{
    for (int64_t i = 0; i < n; ++i) {
        real vn = mu * v[i];
        vn = vn + g[i];
        v[i] = vn;
        real step = lr * vn;
        theta[i] = theta[i] - step;
    }
}

/* ---------------------------------------------------------------------------
 * OptimStep with Adam, the optimiser the paper's experiments use (Section 5.2: "the Adam optimizer with a
 * learning rate of 0.01"; the other constants are not stated and are passed in).  Step t (1-based) of the
 * published algorithm, epsilon added to the root of the bias-corrected second moment:
 *   m <- b1 m + (1 - b1) g;   v <- b2 v + (1 - b2) g^2
 *   theta <- theta - lr * (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps)
 * Each element is computed in double and stored in the storage type.
 * ------------------------------------------------------------------------- */
void so_adam(real *theta, real *m, real *v, const real *g, int64_t n, double lr, double b1, double b2, double eps, int64_t t)
{
    const double c1 = 1.0 - pow(b1, (double)t), c2 = 1.0 - pow(b2, (double)t);
    for (int64_t i = 0; i < n; ++i) {
        const double gi = (double)g[i];
        const double mi = b1 * (double)m[i] + (1.0 - b1) * gi;
        const double vi = b2 * (double)v[i] + (1.0 - b2) * gi * gi;
        m[i] = (real)mi;
        v[i] = (real)vi;
        const double mhat = mi / c1, vhat = vi / c2;
        theta[i] = (real)((double)theta[i] - lr * mhat / (sqrt(vhat) + eps));
    }
}

/* ---------------------------------------------------------------------------
 * ComputeMetric (Algorithm 1): mean IoU of prediction vs. label (Section 3.2):
 *   IoU_c = |pred_c ∩ label_c| / |pred_c ∪ label_c|, averaged over the classes
 *   present in the label.
 * conf[l][q] = #{pixels with label l and prediction q}; pixels whose label or
 * prediction is >= C are skipped and counted in the return value.
 * ------------------------------------------------------------------------- */
int64_t so_confusion(const uint8_t *lab, const uint8_t *pred, int64_t P, int C, int64_t *conf)
{
    int64_t bad = 0;
    memset(conf, 0, sizeof(int64_t) * (size_t)C * C);
    for (int64_t p = 0; p < P; ++p) {
        int l = lab[p], q = pred[p];
        if (l >= C || q >= C) { bad++; continue; }
        conf[(int64_t)l * C + q] += 1;
    }
    return bad;
}

double so_miou(const int64_t *conf, int C)
{
    double sum = 0.0;
    int present = 0;
    for (int c = 0; c < C; ++c) {
        int64_t row = 0, col = 0;
        for (int q = 0; q < C; ++q) { row += conf[(int64_t)c * C + q]; col += conf[(int64_t)q * C + c]; }
        if (row == 0) continue;                 /* class absent from the label */
        int64_t inter = conf[(int64_t)c * C + c];
        sum += (double)inter / (double)(row + col - inter);
        present++;
    }
    return present ? sum / present : 0.0;
}

/* ---------------------------------------------------------------------------
 * Test-only helper: round every element to the nearest bfloat16 value (ties to
 * even), keeping the storage type.  Lets a test separate "wrong" from "rounded"
 * when the CUDA path multiplies bf16 operands.
 * ------------------------------------------------------------------------- */
void so_round_bf16(real *a, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) {
        float f = (float)a[i];
        uint32_t bits;
        memcpy(&bits, &f, 4);
        if ((bits & 0x7f800000u) != 0x7f800000u) {      /* finite */
            uint32_t lsb = (bits >> 16) & 1u;
            bits += 0x7fffu + lsb;
            bits &= 0xffff0000u;
        }
        memcpy(&f, &bits, 4);
        a[i] = (real)f;
    }
}

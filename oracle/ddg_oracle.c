/*
 * ddg_oracle.c — CPU oracle for decoupled parallel backpropagation with delayed gradients (DDG).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference the CUDA library is checked
 * against.  It shares no code, header, table or helper with the CUDA path and nothing in the product
 * path may call it.  Everything is computed in fp64 (the paper does not fix a precision).
 *
 * What it follows in the paper (Huo, Gu, Yang, Huang, ICML 2018):
 *   - Section 2, Eq. 1-5: L-layer feed-forward net h_l = F_l(h_{l-1}; w_l), loss f, forward sweep,
 *     chain-rule backward sweep, SGD.
 *   - Section 3.1, Eq. 6-7: the net is cut into K groups of consecutive layers; at iteration t module k
 *     runs the backward sweep of iteration s = t-K+k, at the weights w^s, on the stale error gradient it
 *     has in store, and hands the error gradient of its input to module k-1 for the next iteration.
 *   - Section 3.3, Eq. 8-9 and Algorithm 1 (SGD-DDG): the delayed gradient is zero while s < 0; every
 *     module updates its own weights with its delayed gradient.  Algorithm 2 (Adam-DDG): the same
 *     delayed gradient feeds Adam moments, bias-corrected with the global iteration count t+1.
 *
 * Readings where the paper is silent (each one is also listed in the design notes of the repository):
 *   - layer formulas: 3x3 cross-correlation, pad 1, no bias; train-mode batch normalisation over
 *     (N,H,W) with biased variance and eps 1e-5; post-activation basic residual block
 *     out = relu(bn2(conv2(relu(bn1(conv1(x))))) + sc(x)); parameter-free shortcut
 *     sc(x)[n,c,h,w] = x[n,c,s*h,s*w] for c < Cin and 0 for the added channels; global mean pool;
 *     fully connected head with bias; mean softmax cross-entropy; relu'(0) = 0.
 *   - ORC_BASIC_BLOCK_PROJ is the same block with a projection shortcut in place of the parameter-free one:
 *     sc(x) = W_s x as a 1x1 convolution with the block's stride, no bias and no batch norm (the paper only
 *     says "ResNet"; this is the plain linear projection of the residual-learning formulation, taken as a second
 *     workload).  Its weight W_s [Cout][Cin] follows bn2.beta in the flat parameter order.
 *   - minibatch loss and gradients are means over the batch.
 *   - momentum / weight decay: d = g + wd*w ; v = mu*v + d ; w = w - lr*v.
 *   - during a module's warm-up (s < 0) nothing at all is applied to it (flag ORC_WARMUP_DECAY
 *     switches to the literal "gradient = 0" update, which still decays and moves momentum).
 *   - the backward sweep of module k differentiates at the stored weights w^s (flag
 *     ORC_USE_CURRENT_WEIGHTS switches to the current weights, the other possible reading).
 *   - flags ORC_ROUND_BF16 / ORC_ROUND_FP32 imitate a storage format: every tensor a sweep stores
 *     (activations, error gradients) and the weights the sweeps read are rounded to bfloat16 or to
 *     float (round to nearest even); batch statistics, logits, loss, parameter gradients, master
 *     weights and optimiser state are rounded to float in both.  All arithmetic between two stores
 *     stays fp64.  This separates format error from mistakes, and it makes the ReLU decisions of a
 *     path that stores the same formats agree with the oracle's.
 *
 * Parity pins (tests/test_oracle_*.py): finite differences, closed forms for softmax-CE and batch
 * norm, brute-force convolution, K=1 == plain backprop, delayed gradient == true gradient at the
 * snapshot, warm-up invariance, lr=0 invariance, an independent library autograd on the same nets.
 * Unpinned by the paper (choices, consistent on both sides): layer formulas, momentum formula, warm-up
 * rule, initialisation, split positions.
 *
 * Tensor layout: NCHW, row-major, fp64.  Flat parameter order: layers in network order; per layer the
 * conv / FC weight ([Cout][Cin][3][3] or [out][in]), then bias, then BN gamma, then BN beta; a basic
 * block contributes conv1.w, bn1.gamma, bn1.beta, conv2.w, bn2.gamma, bn2.beta.
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_FC = 0, ORC_CONV3X3 = 1, ORC_BN = 2, ORC_RELU = 3, ORC_BASIC_BLOCK = 4, ORC_GLOBAL_AVGPOOL = 5,
       ORC_BASIC_BLOCK_PROJ = 6 };
enum { ORC_SGD = 0, ORC_ADAM = 1 };
enum { ORC_USE_CURRENT_WEIGHTS = 1, ORC_WARMUP_DECAY = 2, ORC_ROUND_BF16 = 4, ORC_ROUND_FP32 = 8 };

typedef struct { int kind, c_in, c_out, stride, has_bias, relu_after; } orc_layer;

#define BN_EPS 1e-5

/* ------------------------------------------------------------------------------------------------ */
/* primitives (Section 2, Eq. 3-5 instantiated per layer type)                                      */
/* ------------------------------------------------------------------------------------------------ */

static double *dalloc(size_t n) {
    double *p = (double *)calloc(n ? n : 1, sizeof(double));
    if (!p) { fprintf(stderr, "ddg_oracle: out of memory\n"); abort(); }
    return p;
}

/* y[b][o] = sum_i W[o][i] x[b][i] + bias[o] */
void orc_fc_forward(int B, int in, int out, const double *x, const double *W, const double *bias, double *y) {
    for (int b = 0; b < B; ++b)
        for (int o = 0; o < out; ++o) {
            double acc = bias ? bias[o] : 0.0;
            for (int i = 0; i < in; ++i) acc += W[(size_t)o * in + i] * x[(size_t)b * in + i];
            y[(size_t)b * out + o] = acc;
        }
}

/* dx = dy W ; dW = dy^T x ; db = column sums of dy */
void orc_fc_backward(int B, int in, int out, const double *x, const double *W, const double *dy,
                     double *dx, double *dW, double *db) {
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < in; ++i) {
            double acc = 0.0;
            for (int o = 0; o < out; ++o) acc += dy[(size_t)b * out + o] * W[(size_t)o * in + i];
            dx[(size_t)b * in + i] = acc;
        }
    for (int o = 0; o < out; ++o) {
        for (int i = 0; i < in; ++i) {
            double acc = 0.0;
            for (int b = 0; b < B; ++b) acc += dy[(size_t)b * out + o] * x[(size_t)b * in + i];
            dW[(size_t)o * in + i] = acc;
        }
        if (db) {
            double acc = 0.0;
            for (int b = 0; b < B; ++b) acc += dy[(size_t)b * out + o];
            db[o] = acc;
        }
    }
}

/* y[n][co][ho][wo] = sum_{ci,ky,kx} w[co][ci][ky][kx] * x[n][ci][s*ho+ky-1][s*wo+kx-1], zero outside */
void orc_conv3x3_forward(int B, int Cin, int H, int W, int Cout, int stride, const double *x, const double *w,
                         double *y) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < B; ++n)
        for (int co = 0; co < Cout; ++co) {
            double *yp = y + ((size_t)n * Cout + co) * Ho * Wo;
            for (int i = 0; i < Ho * Wo; ++i) yp[i] = 0.0;
            for (int ci = 0; ci < Cin; ++ci) {
                const double *xp = x + ((size_t)n * Cin + ci) * H * W;
                const double *wp = w + ((size_t)co * Cin + ci) * 9;
                for (int ky = 0; ky < 3; ++ky)
                    for (int kx = 0; kx < 3; ++kx) {
                        const double wv = wp[ky * 3 + kx];
                        for (int ho = 0; ho < Ho; ++ho) {
                            const int hi = stride * ho + ky - 1;
                            if (hi < 0 || hi >= H) continue;
                            for (int wo = 0; wo < Wo; ++wo) {
                                const int wi = stride * wo + kx - 1;
                                if (wi < 0 || wi >= W) continue;
                                yp[ho * Wo + wo] += wv * xp[hi * W + wi];
                            }
                        }
                    }
            }
        }
}

/* dx[n][ci][hi][wi] = sum over (co,ky,kx,ho,wo) hitting that input of w*dy ; dw = sum over (n,ho,wo) of dy*x */
void orc_conv3x3_backward(int B, int Cin, int H, int W, int Cout, int stride, const double *x, const double *w,
                          const double *dy, double *dx, double *dw) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    if (dx) {
#pragma omp parallel for collapse(2) schedule(static)
        for (int n = 0; n < B; ++n)
            for (int ci = 0; ci < Cin; ++ci) {
                double *dxp = dx + ((size_t)n * Cin + ci) * H * W;
                for (int i = 0; i < H * W; ++i) dxp[i] = 0.0;
                for (int co = 0; co < Cout; ++co) {
                    const double *dyp = dy + ((size_t)n * Cout + co) * Ho * Wo;
                    const double *wp = w + ((size_t)co * Cin + ci) * 9;
                    for (int ky = 0; ky < 3; ++ky)
                        for (int kx = 0; kx < 3; ++kx) {
                            const double wv = wp[ky * 3 + kx];
                            for (int ho = 0; ho < Ho; ++ho) {
                                const int hi = stride * ho + ky - 1;
                                if (hi < 0 || hi >= H) continue;
                                for (int wo = 0; wo < Wo; ++wo) {
                                    const int wi = stride * wo + kx - 1;
                                    if (wi < 0 || wi >= W) continue;
                                    dxp[hi * W + wi] += wv * dyp[ho * Wo + wo];
                                }
                            }
                        }
                }
            }
    }
    if (dw) {
#pragma omp parallel for collapse(2) schedule(static)
        for (int co = 0; co < Cout; ++co)
            for (int ci = 0; ci < Cin; ++ci)
                for (int ky = 0; ky < 3; ++ky)
                    for (int kx = 0; kx < 3; ++kx) {
                        double acc = 0.0;
                        for (int n = 0; n < B; ++n) {
                            const double *xp = x + ((size_t)n * Cin + ci) * H * W;
                            const double *dyp = dy + ((size_t)n * Cout + co) * Ho * Wo;
                            for (int ho = 0; ho < Ho; ++ho) {
                                const int hi = stride * ho + ky - 1;
                                if (hi < 0 || hi >= H) continue;
                                for (int wo = 0; wo < Wo; ++wo) {
                                    const int wi = stride * wo + kx - 1;
                                    if (wi < 0 || wi >= W) continue;
                                    acc += dyp[ho * Wo + wo] * xp[hi * W + wi];
                                }
                            }
                        }
                        dw[(((size_t)co * Cin + ci) * 3 + ky) * 3 + kx] = acc;
                    }
    }
}

/* train-mode batch norm over (N, HW): mean, biased variance, y = gamma*(x-mean)*invstd + beta */
void orc_bn_forward(int B, int C, int HW, const double *x, const double *gamma, const double *beta, double *y,
                    double *mean, double *invstd) {
    const double cnt = (double)B * HW;
#pragma omp parallel for schedule(static)
    for (int c = 0; c < C; ++c) {
        double s = 0.0;
        for (int n = 0; n < B; ++n) {
            const double *xp = x + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) s += xp[i];
        }
        const double m = s / cnt;
        double v = 0.0;
        for (int n = 0; n < B; ++n) {
            const double *xp = x + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) v += (xp[i] - m) * (xp[i] - m);
        }
        const double is = 1.0 / sqrt(v / cnt + BN_EPS);
        mean[c] = m;
        invstd[c] = is;
        for (int n = 0; n < B; ++n) {
            const double *xp = x + ((size_t)n * C + c) * HW;
            double *yp = y + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) yp[i] = gamma[c] * (xp[i] - m) * is + beta[c];
        }
    }
}

/* dbeta = sum dy ; dgamma = sum dy*xhat ; dx = gamma*invstd*(dy - dbeta/cnt - xhat*dgamma/cnt) */
void orc_bn_backward(int B, int C, int HW, const double *x, const double *mean, const double *invstd,
                     const double *gamma, const double *dy, double *dx, double *dgamma, double *dbeta) {
    const double cnt = (double)B * HW;
#pragma omp parallel for schedule(static)
    for (int c = 0; c < C; ++c) {
        double sb = 0.0, sg = 0.0;
        for (int n = 0; n < B; ++n) {
            const double *xp = x + ((size_t)n * C + c) * HW;
            const double *dp = dy + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) {
                sb += dp[i];
                sg += dp[i] * (xp[i] - mean[c]) * invstd[c];
            }
        }
        dbeta[c] = sb;
        dgamma[c] = sg;
        for (int n = 0; n < B; ++n) {
            const double *xp = x + ((size_t)n * C + c) * HW;
            const double *dp = dy + ((size_t)n * C + c) * HW;
            double *dxp = dx + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) {
                const double xh = (xp[i] - mean[c]) * invstd[c];
                dxp[i] = gamma[c] * invstd[c] * (dp[i] - sb / cnt - xh * sg / cnt);
            }
        }
    }
}

/* the normalisation alone, from given statistics (used when the statistics were rounded for storage) */
void orc_bn_apply(int B, int C, int HW, const double *x, const double *gamma, const double *beta, const double *mean,
                  const double *invstd, double *y) {
    for (int c = 0; c < C; ++c)
        for (int n = 0; n < B; ++n) {
            const double *xp = x + ((size_t)n * C + c) * HW;
            double *yp = y + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) yp[i] = gamma[c] * (xp[i] - mean[c]) * invstd[c] + beta[c];
        }
}

/* the input gradient alone, from given (possibly storage-rounded) dgamma / dbeta */
void orc_bn_backward_apply(int B, int C, int HW, const double *x, const double *mean, const double *invstd,
                           const double *gamma, const double *dy, const double *dgamma, const double *dbeta,
                           double *dx) {
    const double cnt = (double)B * HW;
    for (int c = 0; c < C; ++c)
        for (int n = 0; n < B; ++n) {
            const double *xp = x + ((size_t)n * C + c) * HW;
            const double *dp = dy + ((size_t)n * C + c) * HW;
            double *dxp = dx + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) {
                const double xh = (xp[i] - mean[c]) * invstd[c];
                dxp[i] = gamma[c] * invstd[c] * (dp[i] - dbeta[c] / cnt - xh * dgamma[c] / cnt);
            }
        }
}

void orc_relu_forward(size_t n, const double *x, double *y) {
    for (size_t i = 0; i < n; ++i) y[i] = x[i] > 0.0 ? x[i] : 0.0;
}

/* y is the relu output; the derivative at 0 is taken as 0 */
void orc_relu_backward(size_t n, const double *y, const double *dy, double *dx) {
    for (size_t i = 0; i < n; ++i) dx[i] = y[i] > 0.0 ? dy[i] : 0.0;
}

/* 1x1 convolution with a spatial stride, no padding, no bias (projection shortcut):
 * y[n,co,ho,wo] = sum_ci w[co][ci] * x[n,ci,stride*ho,stride*wo] */
void orc_conv1x1_forward(int B, int Cin, int H, int W, int Cout, int stride, const double *x, const double *w,
                         double *y) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
#pragma omp parallel for collapse(2)
    for (int n = 0; n < B; ++n)
        for (int co = 0; co < Cout; ++co)
            for (int ho = 0; ho < Ho; ++ho)
                for (int wo = 0; wo < Wo; ++wo) {
                    double acc = 0.0;
                    for (int ci = 0; ci < Cin; ++ci)
                        acc += w[(size_t)co * Cin + ci] * x[(((size_t)n * Cin + ci) * H + stride * ho) * W + stride * wo];
                    y[(((size_t)n * Cout + co) * Ho + ho) * Wo + wo] = acc;
                }
}

/* dx[n,ci,stride*ho,stride*wo] = sum_co w[co][ci] * dy[n,co,ho,wo] (zero at the pixels the stride skips);
 * dw[co][ci] = sum_{n,ho,wo} dy[n,co,ho,wo] * x[n,ci,stride*ho,stride*wo] */
void orc_conv1x1_backward(int B, int Cin, int H, int W, int Cout, int stride, const double *x, const double *w,
                          const double *dy, double *dx, double *dw) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    memset(dx, 0, sizeof(double) * (size_t)B * Cin * H * W);
#pragma omp parallel for collapse(2)
    for (int n = 0; n < B; ++n)
        for (int ci = 0; ci < Cin; ++ci)
            for (int ho = 0; ho < Ho; ++ho)
                for (int wo = 0; wo < Wo; ++wo) {
                    double acc = 0.0;
                    for (int co = 0; co < Cout; ++co)
                        acc += w[(size_t)co * Cin + ci] * dy[(((size_t)n * Cout + co) * Ho + ho) * Wo + wo];
                    dx[(((size_t)n * Cin + ci) * H + stride * ho) * W + stride * wo] = acc;
                }
#pragma omp parallel for collapse(2)
    for (int co = 0; co < Cout; ++co)
        for (int ci = 0; ci < Cin; ++ci) {
            double acc = 0.0;
            for (int n = 0; n < B; ++n)
                for (int ho = 0; ho < Ho; ++ho)
                    for (int wo = 0; wo < Wo; ++wo)
                        acc += dy[(((size_t)n * Cout + co) * Ho + ho) * Wo + wo] *
                               x[(((size_t)n * Cin + ci) * H + stride * ho) * W + stride * wo];
            dw[(size_t)co * Cin + ci] = acc;
        }
}

/* parameter-free shortcut: spatial subsampling by `stride`, new channels are zero */
void orc_shortcut_forward(int B, int Cin, int H, int W, int Cout, int stride, const double *x, double *y) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    for (int n = 0; n < B; ++n)
        for (int c = 0; c < Cout; ++c)
            for (int ho = 0; ho < Ho; ++ho)
                for (int wo = 0; wo < Wo; ++wo)
                    y[(((size_t)n * Cout + c) * Ho + ho) * Wo + wo] =
                        c < Cin ? x[(((size_t)n * Cin + c) * H + stride * ho) * W + stride * wo] : 0.0;
}

void orc_shortcut_backward(int B, int Cin, int H, int W, int Cout, int stride, const double *dy, double *dx) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    memset(dx, 0, sizeof(double) * (size_t)B * Cin * H * W);
    for (int n = 0; n < B; ++n)
        for (int c = 0; c < Cin && c < Cout; ++c)
            for (int ho = 0; ho < Ho; ++ho)
                for (int wo = 0; wo < Wo; ++wo)
                    dx[(((size_t)n * Cin + c) * H + stride * ho) * W + stride * wo] =
                        dy[(((size_t)n * Cout + c) * Ho + ho) * Wo + wo];
}

void orc_avgpool_forward(int B, int C, int HW, const double *x, double *y) {
    for (int i = 0; i < B * C; ++i) {
        double s = 0.0;
        for (int j = 0; j < HW; ++j) s += x[(size_t)i * HW + j];
        y[i] = s / HW;
    }
}

void orc_avgpool_backward(int B, int C, int HW, const double *dy, double *dx) {
    for (int i = 0; i < B * C; ++i)
        for (int j = 0; j < HW; ++j) dx[(size_t)i * HW + j] = dy[i] / HW;
}

/* mean over the batch of -log softmax(z)[y]; dz = (softmax(z) - onehot(y)) / B   (Eq. 1 with f = CE) */
void orc_softmax_ce(int B, int C, const double *z, const int *y, double *loss, double *dz) {
    double total = 0.0;
    for (int b = 0; b < B; ++b) {
        const double *zb = z + (size_t)b * C;
        double mx = zb[0];
        for (int c = 1; c < C; ++c) if (zb[c] > mx) mx = zb[c];
        double se = 0.0;
        for (int c = 0; c < C; ++c) se += exp(zb[c] - mx);
        total += log(se) + mx - zb[y[b]];
        if (dz)
            for (int c = 0; c < C; ++c)
                dz[(size_t)b * C + c] = (exp(zb[c] - mx) / se - (c == y[b] ? 1.0 : 0.0)) / B;
    }
    *loss = total / B;
}

/* round to nearest even onto the bfloat16 grid, via fp32 as the CUDA path's arithmetic does */
static double bf16_round(double v) {
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return (double)f; /* inf / nan pass through */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return (double)f;
}

double orc_bf16_round(double v) { return bf16_round(v); }

/* ------------------------------------------------------------------------------------------------ */
/* the network: layers, modules, per-sample history                                                 */
/* ------------------------------------------------------------------------------------------------ */

typedef struct {
    orc_layer spec;
    int C_in, H_in, W_in;    /* input tensor is [B][C_in][H_in][W_in] */
    int C_out, H_out, W_out; /* output tensor */
    size_t p_off, p_cnt;     /* slice of the flat parameter vector */
    int module;              /* 0-based group index */
} layer_t;

/* everything one layer's forward sweep keeps for its backward sweep (Eq. 6-7 need h^{s} of every layer) */
typedef struct {
    double *x;   /* layer input */
    double *y;   /* layer output (after the optional relu) */
    double *y1, *a1, *y2;          /* basic block: conv1 out, relu(bn1), conv2 out */
    double *m1, *is1, *m2, *is2;   /* batch statistics (bn layer uses m1/is1) */
} cache_t;

typedef struct {
    int s;            /* iteration this record belongs to, -1 = empty */
    double *w;        /* snapshot w^s of this module's parameter slice */
    cache_t *caches;  /* one per layer of the module */
    double *delta;    /* error gradient w.r.t. the module output for sample s, once known */
    int has_delta;
} hist_t;

typedef struct {
    int n_layers, K, B, num_classes, flags;
    int in_c, in_h, in_w;
    layer_t *layers;
    int *first, *last;      /* layer range [first,last] of each module */
    size_t *m_off, *m_cnt;  /* parameter slice of each module */
    size_t P;
    double *w;              /* current weights w^t */
    double *v, *m2nd;       /* optimiser state: momentum / Adam first moment in v, second moment in m2nd */
    double *g;              /* last applied delayed gradients, flat; */
    int *g_valid, *g_sample;
    int opt;
    double lr, mu, wd, b1, b2, eps;
    long t;
    int n_hist;             /* K+1 records per module */
    hist_t **hist;          /* hist[k][slot] */
    int **labels_hist;      /* labels of the in-flight iterations */
    long *labels_s;
} orc_ctx;

static size_t tsize(const orc_ctx *c, int C, int H, int W) { return (size_t)c->B * C * H * W; }

/* storage rounding of activations, error gradients and sweep weights */
static void maybe_round(const orc_ctx *c, double *p, size_t n) {
    if (c->flags & ORC_ROUND_BF16) for (size_t i = 0; i < n; ++i) p[i] = bf16_round(p[i]);
    else if (c->flags & ORC_ROUND_FP32) for (size_t i = 0; i < n; ++i) p[i] = (double)(float)p[i];
}

/* storage rounding of what is kept in float in both formats */
static void maybe_round32(const orc_ctx *c, double *p, size_t n) {
    if (c->flags & (ORC_ROUND_BF16 | ORC_ROUND_FP32)) for (size_t i = 0; i < n; ++i) p[i] = (double)(float)p[i];
}

/* batch norm forward with the statistics passing through storage */
static void bn_forward_stored(const orc_ctx *c, int B, int C, int HW, const double *x, const double *gamma,
                              const double *beta, double *y, double *mean, double *invstd) {
    orc_bn_forward(B, C, HW, x, gamma, beta, y, mean, invstd);
    if (c->flags & (ORC_ROUND_BF16 | ORC_ROUND_FP32)) {
        maybe_round32(c, mean, C); maybe_round32(c, invstd, C);
        orc_bn_apply(B, C, HW, x, gamma, beta, mean, invstd, y);
    }
}

/* batch norm backward with dgamma / dbeta passing through storage */
static void bn_backward_stored(const orc_ctx *c, int B, int C, int HW, const double *x, const double *mean,
                               const double *invstd, const double *gamma, const double *dy, double *dx,
                               double *dgamma, double *dbeta) {
    orc_bn_backward(B, C, HW, x, mean, invstd, gamma, dy, dx, dgamma, dbeta);
    if (c->flags & (ORC_ROUND_BF16 | ORC_ROUND_FP32)) {
        maybe_round32(c, dgamma, C); maybe_round32(c, dbeta, C);
        orc_bn_backward_apply(B, C, HW, x, mean, invstd, gamma, dy, dgamma, dbeta, dx);
    }
}

static void free_cache(cache_t *q) {
    free(q->x); free(q->y); free(q->y1); free(q->a1); free(q->y2);
    free(q->m1); free(q->is1); free(q->m2); free(q->is2);
    memset(q, 0, sizeof(*q));
}

static double *dup(const double *src, size_t n) {
    double *p = dalloc(n);
    memcpy(p, src, n * sizeof(double));
    return p;
}

/* forward sweep of one layer (Eq. 3).  `w` points at the layer's own parameter slice.  Returns the
 * freshly allocated output; fills `q` with what the backward sweep needs. */
static double *layer_forward(orc_ctx *c, const layer_t *L, const double *w, const double *x, cache_t *q) {
    const int B = c->B;
    const size_t n_in = tsize(c, L->C_in, L->H_in, L->W_in), n_out = tsize(c, L->C_out, L->H_out, L->W_out);
    const int is_last = (L == &c->layers[c->n_layers - 1]);
    double *y = dalloc(n_out);
    q->x = dup(x, n_in);
    switch (L->spec.kind) {
    case ORC_FC:
        orc_fc_forward(B, L->C_in, L->C_out, x, w, L->spec.has_bias ? w + (size_t)L->C_in * L->C_out : NULL, y);
        if (L->spec.relu_after) orc_relu_forward(n_out, y, y);
        if (!is_last) maybe_round(c, y, n_out);
        else maybe_round32(c, y, n_out); /* the network output (logits) is kept in float */
        break;
    case ORC_CONV3X3:
        orc_conv3x3_forward(B, L->C_in, L->H_in, L->W_in, L->C_out, L->spec.stride, x, w, y);
        if (L->spec.relu_after) orc_relu_forward(n_out, y, y);
        maybe_round(c, y, n_out);
        break;
    case ORC_BN:
        q->m1 = dalloc(L->C_in); q->is1 = dalloc(L->C_in);
        bn_forward_stored(c, B, L->C_in, L->H_in * L->W_in, x, w, w + L->C_in, y, q->m1, q->is1);
        if (L->spec.relu_after) orc_relu_forward(n_out, y, y);
        maybe_round(c, y, n_out);
        break;
    case ORC_RELU:
        orc_relu_forward(n_out, x, y);
        break;
    case ORC_GLOBAL_AVGPOOL:
        orc_avgpool_forward(B, L->C_in, L->H_in * L->W_in, x, y);
        maybe_round(c, y, n_out);
        break;
    case ORC_BASIC_BLOCK:
    case ORC_BASIC_BLOCK_PROJ: {
        const int Ci = L->C_in, Co = L->C_out, st = L->spec.stride;
        const double *w1 = w, *g1 = w1 + (size_t)Co * Ci * 9, *b1 = g1 + Co;
        const double *w2 = b1 + Co, *g2 = w2 + (size_t)Co * Co * 9, *b2 = g2 + Co, *ws = b2 + Co;
        const int HWo = L->H_out * L->W_out;
        q->y1 = dalloc(n_out); q->a1 = dalloc(n_out); q->y2 = dalloc(n_out);
        q->m1 = dalloc(Co); q->is1 = dalloc(Co); q->m2 = dalloc(Co); q->is2 = dalloc(Co);
        orc_conv3x3_forward(B, Ci, L->H_in, L->W_in, Co, st, x, w1, q->y1);
        maybe_round(c, q->y1, n_out);
        bn_forward_stored(c, B, Co, HWo, q->y1, g1, b1, q->a1, q->m1, q->is1);
        orc_relu_forward(n_out, q->a1, q->a1);
        maybe_round(c, q->a1, n_out);
        orc_conv3x3_forward(B, Co, L->H_out, L->W_out, Co, 1, q->a1, w2, q->y2);
        maybe_round(c, q->y2, n_out);
        double *z = dalloc(n_out), *sc = dalloc(n_out);
        bn_forward_stored(c, B, Co, HWo, q->y2, g2, b2, z, q->m2, q->is2);
        if (L->spec.kind == ORC_BASIC_BLOCK_PROJ) {
            orc_conv1x1_forward(B, Ci, L->H_in, L->W_in, Co, st, x, ws, sc);
            maybe_round(c, sc, n_out); /* the projected shortcut is a stored tensor */
        } else {
            orc_shortcut_forward(B, Ci, L->H_in, L->W_in, Co, st, x, sc);
        }
        for (size_t i = 0; i < n_out; ++i) z[i] += sc[i];
        orc_relu_forward(n_out, z, y);
        maybe_round(c, y, n_out);
        free(z); free(sc);
        break;
    }
    default: abort();
    }
    q->y = dup(y, n_out);
    return y;
}

/* backward sweep of one layer (Eq. 4-5, or Eq. 6-7 when the cache and weights are stale ones).
 * dy is consumed; returns dx (freshly allocated); writes this layer's parameter gradient to gw. */
static double *layer_backward(const orc_ctx *c, const layer_t *L, const double *w, const cache_t *q,
                              const double *dy_in, double *gw) {
    const int B = c->B;
    const size_t n_in = tsize(c, L->C_in, L->H_in, L->W_in), n_out = tsize(c, L->C_out, L->H_out, L->W_out);
    const int is_first = (L == &c->layers[0]);
    double *dx = dalloc(n_in);
    double *dy = dup(dy_in, n_out);
    switch (L->spec.kind) {
    case ORC_FC:
        if (L->spec.relu_after) orc_relu_backward(n_out, q->y, dy, dy);
        orc_fc_backward(B, L->C_in, L->C_out, q->x, w, dy, dx, gw,
                        L->spec.has_bias ? gw + (size_t)L->C_in * L->C_out : NULL);
        break;
    case ORC_CONV3X3:
        if (L->spec.relu_after) orc_relu_backward(n_out, q->y, dy, dy);
        orc_conv3x3_backward(B, L->C_in, L->H_in, L->W_in, L->C_out, L->spec.stride, q->x, w, dy, dx, gw);
        break;
    case ORC_BN:
        if (L->spec.relu_after) orc_relu_backward(n_out, q->y, dy, dy);
        bn_backward_stored(c, B, L->C_in, L->H_in * L->W_in, q->x, q->m1, q->is1, w, dy, dx, gw, gw + L->C_in);
        break;
    case ORC_RELU:
        orc_relu_backward(n_out, q->y, dy, dx);
        break;
    case ORC_GLOBAL_AVGPOOL:
        orc_avgpool_backward(B, L->C_in, L->H_in * L->W_in, dy, dx);
        break;
    case ORC_BASIC_BLOCK:
    case ORC_BASIC_BLOCK_PROJ: {
        const int Ci = L->C_in, Co = L->C_out, st = L->spec.stride;
        const size_t nw1 = (size_t)Co * Ci * 9, nw2 = (size_t)Co * Co * 9;
        const double *w1 = w, *g1 = w1 + nw1, *w2 = g1 + 2 * Co, *g2 = w2 + nw2, *ws = g2 + 2 * Co;
        double *gw1 = gw, *gg1 = gw1 + nw1, *gb1 = gg1 + Co, *gw2 = gb1 + Co, *gg2 = gw2 + nw2, *gb2 = gg2 + Co;
        const int HWo = L->H_out * L->W_out;
        double *dz = dalloc(n_out), *dy2 = dalloc(n_out), *da1 = dalloc(n_out), *dy1 = dalloc(n_out);
        double *dsc = dalloc(n_in);
        orc_relu_backward(n_out, q->y, dy, dz);               /* through the final relu */
        bn_backward_stored(c, B, Co, HWo, q->y2, q->m2, q->is2, g2, dz, dy2, gg2, gb2);
        maybe_round(c, dy2, n_out);
        orc_conv3x3_backward(B, Co, L->H_out, L->W_out, Co, 1, q->a1, w2, dy2, da1, gw2);
        maybe_round(c, da1, n_out);
        orc_relu_backward(n_out, q->a1, da1, da1);
        bn_backward_stored(c, B, Co, HWo, q->y1, q->m1, q->is1, g1, da1, dy1, gg1, gb1);
        maybe_round(c, dy1, n_out);
        orc_conv3x3_backward(B, Ci, L->H_in, L->W_in, Co, st, q->x, w1, dy1, dx, gw1);
        if (L->spec.kind == ORC_BASIC_BLOCK_PROJ)
            orc_conv1x1_backward(B, Ci, L->H_in, L->W_in, Co, st, q->x, ws, dz, dsc, gb2 + Co);
        else
            orc_shortcut_backward(B, Ci, L->H_in, L->W_in, Co, st, dz, dsc);
        for (size_t i = 0; i < n_in; ++i) dx[i] += dsc[i];
        free(dz); free(dy2); free(da1); free(dy1); free(dsc);
        break;
    }
    default: abort();
    }
    if (!is_first) maybe_round(c, dx, n_in);
    maybe_round32(c, gw, L->p_cnt); /* parameter gradients are kept in float */
    free(dy);
    return dx;
}

static size_t layer_param_count(const orc_layer *s) {
    switch (s->kind) {
    case ORC_FC: return (size_t)s->c_in * s->c_out + (s->has_bias ? s->c_out : 0);
    case ORC_CONV3X3: return (size_t)s->c_in * s->c_out * 9;
    case ORC_BN: return 2 * (size_t)s->c_in;
    case ORC_BASIC_BLOCK: return (size_t)s->c_in * s->c_out * 9 + (size_t)s->c_out * s->c_out * 9 + 4 * (size_t)s->c_out;
    case ORC_BASIC_BLOCK_PROJ:
        return (size_t)s->c_in * s->c_out * 9 + (size_t)s->c_out * s->c_out * 9 + 4 * (size_t)s->c_out + (size_t)s->c_in * s->c_out;
    default: return 0;
    }
}

void orc_destroy(orc_ctx *c);

orc_ctx *orc_create(const orc_layer *layers, int n_layers, const int *split_after, int K, int opt, double lr,
                    double mu, double wd, double b1, double b2, double eps, int batch, int in_c, int in_h,
                    int in_w, int num_classes, int flags) {
    if (n_layers < 1 || K < 1 || K > n_layers || batch < 1) return NULL;
    orc_ctx *c = (orc_ctx *)calloc(1, sizeof(orc_ctx));
    c->n_layers = n_layers; c->K = K; c->B = batch; c->num_classes = num_classes; c->flags = flags;
    c->in_c = in_c; c->in_h = in_h; c->in_w = in_w;
    c->opt = opt; c->lr = lr; c->mu = mu; c->wd = wd; c->b1 = b1; c->b2 = b2; c->eps = eps;
    c->layers = (layer_t *)calloc(n_layers, sizeof(layer_t));
    int C = in_c, H = in_h, W = in_w;
    size_t off = 0;
    for (int l = 0; l < n_layers; ++l) {
        layer_t *L = &c->layers[l];
        L->spec = layers[l];
        L->C_in = C; L->H_in = H; L->W_in = W;
        int ok = 1;
        switch (layers[l].kind) {
        case ORC_FC: ok = (H == 1 && W == 1 && layers[l].c_in == C); C = layers[l].c_out; break;
        case ORC_CONV3X3:
        case ORC_BASIC_BLOCK:
        case ORC_BASIC_BLOCK_PROJ:
            ok = (layers[l].c_in == C && (layers[l].stride == 1 || layers[l].stride == 2) &&
                  layers[l].c_out >= layers[l].c_in);
            if (layers[l].kind == ORC_BASIC_BLOCK_PROJ) ok = (layers[l].c_in == C && (layers[l].stride == 1 || layers[l].stride == 2));
            if (layers[l].kind == ORC_CONV3X3) ok = (layers[l].c_in == C && (layers[l].stride == 1 || layers[l].stride == 2));
            C = layers[l].c_out; H = (H - 1) / layers[l].stride + 1; W = (W - 1) / layers[l].stride + 1; break;
        case ORC_BN: ok = (layers[l].c_in == C); break;
        case ORC_RELU: break;
        case ORC_GLOBAL_AVGPOOL: H = 1; W = 1; break;
        default: ok = 0;
        }
        if (!ok) { free(c->layers); free(c); return NULL; }
        L->C_out = C; L->H_out = H; L->W_out = W;
        L->p_off = off; L->p_cnt = layer_param_count(&layers[l]);
        off += L->p_cnt;
    }
    if (C != num_classes || H != 1 || W != 1) { free(c->layers); free(c); return NULL; }
    c->P = off;
    c->first = (int *)calloc(K, sizeof(int)); c->last = (int *)calloc(K, sizeof(int));
    c->m_off = (size_t *)calloc(K, sizeof(size_t)); c->m_cnt = (size_t *)calloc(K, sizeof(size_t));
    for (int k = 0; k < K; ++k) {
        c->first[k] = k == 0 ? 0 : split_after[k - 1] + 1;
        c->last[k] = k == K - 1 ? n_layers - 1 : split_after[k];
        if (c->first[k] > c->last[k] || c->last[k] >= n_layers) {
            free(c->first); free(c->last); free(c->m_off); free(c->m_cnt); free(c->layers); free(c); return NULL;
        }
        c->m_off[k] = c->layers[c->first[k]].p_off;
        c->m_cnt[k] = c->layers[c->last[k]].p_off + c->layers[c->last[k]].p_cnt - c->m_off[k];
        for (int l = c->first[k]; l <= c->last[k]; ++l) c->layers[l].module = k;
    }
    c->w = dalloc(c->P); c->v = dalloc(c->P); c->m2nd = dalloc(c->P); c->g = dalloc(c->P);
    c->g_valid = (int *)calloc(K, sizeof(int)); c->g_sample = (int *)calloc(K, sizeof(int));
    c->n_hist = K + 1;
    c->hist = (hist_t **)calloc(K, sizeof(hist_t *));
    for (int k = 0; k < K; ++k) {
        c->hist[k] = (hist_t *)calloc(c->n_hist, sizeof(hist_t));
        for (int j = 0; j < c->n_hist; ++j) {
            c->hist[k][j].s = -1;
            c->hist[k][j].caches = (cache_t *)calloc(c->last[k] - c->first[k] + 1, sizeof(cache_t));
        }
    }
    c->labels_hist = (int **)calloc(c->n_hist, sizeof(int *));
    c->labels_s = (long *)calloc(c->n_hist, sizeof(long));
    for (int j = 0; j < c->n_hist; ++j) { c->labels_hist[j] = (int *)calloc(batch, sizeof(int)); c->labels_s[j] = -1; }
    return c;
}

static void clear_hist(orc_ctx *c, hist_t *h, int k) {
    for (int l = 0; l <= c->last[k] - c->first[k]; ++l) free_cache(&h->caches[l]);
    free(h->w); h->w = NULL;
    free(h->delta); h->delta = NULL;
    h->has_delta = 0;
    h->s = -1;
}

void orc_destroy(orc_ctx *c) {
    if (!c) return;
    for (int k = 0; k < c->K; ++k) {
        for (int j = 0; j < c->n_hist; ++j) { clear_hist(c, &c->hist[k][j], k); free(c->hist[k][j].caches); }
        free(c->hist[k]);
    }
    for (int j = 0; j < c->n_hist; ++j) free(c->labels_hist[j]);
    free(c->labels_hist); free(c->labels_s);
    free(c->hist); free(c->layers); free(c->first); free(c->last); free(c->m_off); free(c->m_cnt);
    free(c->w); free(c->v); free(c->m2nd); free(c->g); free(c->g_valid); free(c->g_sample);
    free(c);
}

size_t orc_param_count(const orc_ctx *c) { return c->P; }
void orc_module_param_counts(const orc_ctx *c, size_t *per_module) {
    for (int k = 0; k < c->K; ++k) per_module[k] = c->m_cnt[k];
}
void orc_set_weights(orc_ctx *c, const double *w) { memcpy(c->w, w, c->P * sizeof(double)); }
void orc_get_weights(const orc_ctx *c, double *w) { memcpy(w, c->w, c->P * sizeof(double)); }
void orc_set_lr(orc_ctx *c, double lr) { c->lr = lr; }
long orc_iteration(const orc_ctx *c) { return c->t; }

/* last applied delayed gradient of module k (0-based).  Returns the sample index s it belongs to, or -1
 * when the module was still in warm-up at the last step (Eq. 8: gradient is zero, dst is zero-filled). */
int orc_get_grads(const orc_ctx *c, int k, double *dst) {
    if (!c->g_valid[k]) { memset(dst, 0, c->m_cnt[k] * sizeof(double)); return -1; }
    memcpy(dst, c->g + c->m_off[k], c->m_cnt[k] * sizeof(double));
    return c->g_sample[k];
}

/* the weights a sweep reads: the given slice, rounded when bf16 storage is being imitated */
static double *sweep_weights(const orc_ctx *c, const double *w, size_t n) {
    double *p = dup(w, n);
    maybe_round(c, p, n);
    return p;
}

/* loss of the whole net at the current weights, no state change (for finite-difference pins) */
double orc_loss_only(orc_ctx *c, const double *x, const int *y) {
    double *h = dup(x, tsize(c, c->in_c, c->in_h, c->in_w));
    maybe_round(c, h, tsize(c, c->in_c, c->in_h, c->in_w));
    for (int l = 0; l < c->n_layers; ++l) {
        cache_t q; memset(&q, 0, sizeof(q));
        double *wl = sweep_weights(c, c->w + c->layers[l].p_off, c->layers[l].p_cnt);
        double *o = layer_forward(c, &c->layers[l], wl, h, &q);
        free(wl); free_cache(&q); free(h);
        h = o;
    }
    double loss;
    orc_softmax_ce(c->B, c->num_classes, h, y, &loss, NULL);
    maybe_round32(c, &loss, 1);
    free(h);
    return loss;
}

/* One DDG iteration t (Algorithm 1 / Algorithm 2 with the backward sweeps of Eq. 6-7). */
double orc_step(orc_ctx *c, const double *x, const int *y) {
    const int K = c->K;
    const long t = c->t;
    const int slot_t = (int)(t % c->n_hist);
    memcpy(c->labels_hist[slot_t], y, c->B * sizeof(int));
    c->labels_s[slot_t] = t;

    /* 1. forward sweep through modules 1..K with the current weights w^t (Eq. 3); keep h^t and w^t */
    double *h = dup(x, tsize(c, c->in_c, c->in_h, c->in_w));
    maybe_round(c, h, tsize(c, c->in_c, c->in_h, c->in_w));
    for (int k = 0; k < K; ++k) {
        hist_t *rec = &c->hist[k][slot_t];
        clear_hist(c, rec, k);
        rec->s = (int)t;
        rec->w = dup(c->w + c->m_off[k], c->m_cnt[k]);
        for (int l = c->first[k]; l <= c->last[k]; ++l) {
            const layer_t *L = &c->layers[l];
            double *wl = sweep_weights(c, c->w + L->p_off, L->p_cnt);
            double *o = layer_forward(c, L, wl, h, &rec->caches[l - c->first[k]]);
            free(wl); free(h);
            h = o;
        }
    }
    /* loss f and its gradient w.r.t. the network output: the up-to-date delta of module K */
    double loss;
    {
        hist_t *rec = &c->hist[K - 1][slot_t];
        rec->delta = dalloc((size_t)c->B * c->num_classes);
        orc_softmax_ce(c->B, c->num_classes, h, y, &loss, rec->delta);
        maybe_round32(c, rec->delta, (size_t)c->B * c->num_classes);
        maybe_round32(c, &loss, 1);
        rec->has_delta = 1;
    }
    free(h);

    /* 2. every module k runs its backward sweep on sample s = t-K+k (k 1-based) with the delta it has in
     *    store; modules are independent of one another within the iteration.  New deltas are parked and
     *    delivered after all modules have run, so that no module sees a delta produced in this iteration
     *    (module K's own loss gradient aside). */
    double **parked = (double **)calloc(K, sizeof(double *));
    for (int k0 = 0; k0 < K; ++k0) {
        const long s = t - K + (k0 + 1);
        c->g_valid[k0] = 0;
        if (s < 0) continue; /* Eq. 8: delayed gradient is zero during warm-up */
        hist_t *rec = &c->hist[k0][(int)(s % c->n_hist)];
        if (rec->s != s || !rec->has_delta) { fprintf(stderr, "ddg_oracle: history miss k=%d s=%ld\n", k0, s); abort(); }
        const double *wsrc = (c->flags & ORC_USE_CURRENT_WEIGHTS) ? c->w + c->m_off[k0] : rec->w;
        double *d = dup(rec->delta, tsize(c, c->layers[c->last[k0]].C_out, c->layers[c->last[k0]].H_out,
                                          c->layers[c->last[k0]].W_out));
        for (int l = c->last[k0]; l >= c->first[k0]; --l) {
            const layer_t *L = &c->layers[l];
            double *wl = sweep_weights(c, wsrc + (L->p_off - c->m_off[k0]), L->p_cnt);
            double *dx = layer_backward(c, L, wl, &rec->caches[l - c->first[k0]], d, c->g + L->p_off);
            free(wl); free(d);
            d = dx;
        }
        c->g_valid[k0] = 1;
        c->g_sample[k0] = (int)s;
        if (k0 > 0) parked[k0] = d; else free(d);
    }
    for (int k0 = 1; k0 < K; ++k0) {
        if (!parked[k0]) continue;
        const long s = t - K + (k0 + 1);
        hist_t *below = &c->hist[k0 - 1][(int)(s % c->n_hist)];
        if (below->s != s) { fprintf(stderr, "ddg_oracle: delta hand-off miss\n"); abort(); }
        free(below->delta);
        below->delta = parked[k0];
        below->has_delta = 1;
    }
    free(parked);

    /* 3. every module updates its own weights with its delayed gradient (Eq. 9) */
    for (int k0 = 0; k0 < K; ++k0) {
        const size_t o = c->m_off[k0], n = c->m_cnt[k0];
        const int have = c->g_valid[k0];
        if (!have && !(c->flags & ORC_WARMUP_DECAY)) continue;
        if (c->opt == ORC_SGD) {
            for (size_t i = o; i < o + n; ++i) {
                const double d = (have ? c->g[i] : 0.0) + c->wd * c->w[i];
                c->v[i] = c->mu * c->v[i] + d;
                c->w[i] -= c->lr * c->v[i];
            }
            maybe_round32(c, c->v + o, n); maybe_round32(c, c->w + o, n);
        } else { /* Algorithm 2: bias correction with the global count t+1 */
            const double c1 = 1.0 - pow(c->b1, (double)(t + 1)), c2 = 1.0 - pow(c->b2, (double)(t + 1));
            for (size_t i = o; i < o + n; ++i) {
                const double gi = have ? c->g[i] : 0.0;
                c->v[i] = c->b1 * c->v[i] + (1.0 - c->b1) * gi;
                c->m2nd[i] = c->b2 * c->m2nd[i] + (1.0 - c->b2) * gi * gi;
                c->w[i] -= c->lr * (c->v[i] / c1) / (sqrt(c->m2nd[i] / c2) + c->eps);
            }
            maybe_round32(c, c->v + o, n); maybe_round32(c, c->m2nd + o, n); maybe_round32(c, c->w + o, n);
        }
    }
    c->t = t + 1;
    return loss;
}

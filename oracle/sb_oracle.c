/*
 * CPU oracle for the SplitBrain hybrid data/model-parallel training step: layer primitives.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA library is
 * checked against.  It shares no code with the CUDA path and is never called by it.
 *
 * Every routine is the textbook definition written as direct loops: no blocking, no im2col,
 * no fusion, no reordering.  OpenMP only distributes *independent outputs* over threads; the
 * summation order inside one output element is fixed and the same for any thread count.
 *
 * Compiled twice: -DREAL=float (the contract precision) and -DREAL=double (used by the
 * finite-difference and closed-form pins).
 *
 * Layouts: activations NHWC; conv weights [Cout][3][3][Cin]; FC weights [out][in].
 *
 * What the paper fixes and what it leaves open (paper section in brackets):
 *  - conv layers are replicated, FC layers are split 1/K by output column, ReLU follows the
 *    partitioned width [Design, Layer Partitioning, Listing 1];
 *  - convolution = 3x3 cross-correlation, stride 1, zero pad 1, one bias per output channel
 *    (the paper specifies a convolutional layer by its kernel and output sizes only; Table 1 counts 9*Cin*Cout weights);
 *  - pooling = 2x2 max, stride 2; ties resolved to the first maximum in scan order
 *    (0,0),(0,1),(1,0),(1,1);  ReLU'(0) = 0;
 *  - loss = log-softmax + negative log-likelihood, mean over the full batch [Listing 1,
 *    LOG_SOFTMAX case];
 *  - SGD with momentum in the Torch form v <- mu*v + g, w <- w - lr*v [Implementation; the constants come
 *    from the benchmark configuration].
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

#ifndef REAL
#define REAL float
#endif

#define IDX4(n, h, w, c, H, W, C) ((((size_t)(n) * (H) + (h)) * (W) + (w)) * (C) + (c))

/* y[n,h,w,k] = act(bias[k] + sum_{r,s,c} x[n,h+r-1,w+s-1,c] * wt[k,r,s,c]), zero outside the image. */
void orc_conv3x3_fwd(const REAL* x, const REAL* wt, const REAL* bias, REAL* y,
                     int N, int H, int W, int Cin, int Cout, int relu)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int h = 0; h < H; ++h)
            for (int w = 0; w < W; ++w)
                for (int k = 0; k < Cout; ++k) {
                    REAL acc = bias[k];
                    for (int r = 0; r < 3; ++r) {
                        int hh = h + r - 1;
                        if (hh < 0 || hh >= H) continue;
                        for (int s = 0; s < 3; ++s) {
                            int ww = w + s - 1;
                            if (ww < 0 || ww >= W) continue;
                            const REAL* xp = x + IDX4(n, hh, ww, 0, H, W, Cin);
                            const REAL* wp = wt + (((size_t)k * 3 + r) * 3 + s) * Cin;
                            for (int c = 0; c < Cin; ++c) acc += xp[c] * wp[c];
                        }
                    }
                    if (relu && !(acc > (REAL)0)) acc = (REAL)0;
                    y[IDX4(n, h, w, k, H, W, Cout)] = acc;
                }
}

/* dx[n,h,w,c] = sum_{r,s,k} dy[n,h-r+1,w-s+1,k] * wt[k,r,s,c]  (terms outside the image are zero). */
void orc_conv3x3_dgrad(const REAL* dy, const REAL* wt, REAL* dx,
                       int N, int H, int W, int Cin, int Cout)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int h = 0; h < H; ++h)
            for (int w = 0; w < W; ++w)
                for (int c = 0; c < Cin; ++c) {
                    REAL acc = (REAL)0;
                    for (int r = 0; r < 3; ++r) {
                        int hh = h - r + 1;
                        if (hh < 0 || hh >= H) continue;
                        for (int s = 0; s < 3; ++s) {
                            int ww = w - s + 1;
                            if (ww < 0 || ww >= W) continue;
                            const REAL* dp = dy + IDX4(n, hh, ww, 0, H, W, Cout);
                            for (int k = 0; k < Cout; ++k)
                                acc += dp[k] * wt[(((size_t)k * 3 + r) * 3 + s) * Cin + c];
                        }
                    }
                    dx[IDX4(n, h, w, c, H, W, Cin)] = acc;
                }
}

/* dw[k,r,s,c] = sum_{n,h,w} dy[n,h,w,k] * x[n,h+r-1,w+s-1,c];  db[k] = sum_{n,h,w} dy[n,h,w,k]. */
void orc_conv3x3_wgrad(const REAL* x, const REAL* dy, REAL* dw, REAL* db,
                       int N, int H, int W, int Cin, int Cout)
{
#pragma omp parallel for schedule(static)
    for (int k = 0; k < Cout; ++k) {
        REAL sb = (REAL)0;
        for (int n = 0; n < N; ++n)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w) sb += dy[IDX4(n, h, w, k, H, W, Cout)];
        db[k] = sb;
        for (int r = 0; r < 3; ++r)
            for (int s = 0; s < 3; ++s)
                for (int c = 0; c < Cin; ++c) {
                    REAL acc = (REAL)0;
                    for (int n = 0; n < N; ++n)
                        for (int h = 0; h < H; ++h) {
                            int hh = h + r - 1;
                            if (hh < 0 || hh >= H) continue;
                            for (int w = 0; w < W; ++w) {
                                int ww = w + s - 1;
                                if (ww < 0 || ww >= W) continue;
                                acc += dy[IDX4(n, h, w, k, H, W, Cout)] * x[IDX4(n, hh, ww, c, H, W, Cin)];
                            }
                        }
                    dw[(((size_t)k * 3 + r) * 3 + s) * Cin + c] = acc;
                }
    }
}

/* p = max over the 2x2 window; idx in {0,1,2,3} = position (dh*2+dw) of the first maximum. */
void orc_maxpool2_fwd(const REAL* x, REAL* p, uint8_t* idx, int N, int H, int W, int C)
{
    int Ho = H / 2, Wo = W / 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int h = 0; h < Ho; ++h)
            for (int w = 0; w < Wo; ++w)
                for (int c = 0; c < C; ++c) {
                    REAL best = x[IDX4(n, 2 * h, 2 * w, c, H, W, C)];
                    uint8_t bi = 0;
                    for (int q = 1; q < 4; ++q) {
                        REAL v = x[IDX4(n, 2 * h + (q >> 1), 2 * w + (q & 1), c, H, W, C)];
                        if (v > best) { best = v; bi = (uint8_t)q; }
                    }
                    p[IDX4(n, h, w, c, Ho, Wo, C)] = best;
                    idx[IDX4(n, h, w, c, Ho, Wo, C)] = bi;
                }
}

/* dx = dp routed to the recorded argmax position, zero elsewhere. */
void orc_maxpool2_bwd(const REAL* dp, const uint8_t* idx, REAL* dx, int N, int H, int W, int C)
{
    int Ho = H / 2, Wo = W / 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int h = 0; h < Ho; ++h)
            for (int w = 0; w < Wo; ++w)
                for (int c = 0; c < C; ++c) {
                    size_t o = IDX4(n, h, w, c, Ho, Wo, C);
                    for (int q = 0; q < 4; ++q)
                        dx[IDX4(n, 2 * h + (q >> 1), 2 * w + (q & 1), c, H, W, C)] =
                            (q == idx[o]) ? dp[o] : (REAL)0;
                }
}

/* One column shard of an FC layer: Y[g,o] = act(b[o] + sum_i X[g,i] * Wt[o,i]), o in [0,out_j). */
void orc_fc_fwd(const REAL* X, const REAL* Wt, const REAL* b, REAL* Y,
                int B, int in, int out_j, int relu)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int g = 0; g < B; ++g)
        for (int o = 0; o < out_j; ++o) {
            REAL acc = b[o];
            const REAL* xp = X + (size_t)g * in;
            const REAL* wp = Wt + (size_t)o * in;
            for (int i = 0; i < in; ++i) acc += xp[i] * wp[i];
            if (relu && !(acc > (REAL)0)) acc = (REAL)0;
            Y[(size_t)g * out_j + o] = acc;
        }
}

/* Shard backward: dW[o,i] = sum_g dY[g,o]*X[g,i];  db[o] = sum_g dY[g,o];
 * dX[g,i] = sum_o dY[g,o]*Wt[o,i]  (this shard's contribution to the full-width input gradient). */
void orc_fc_bwd(const REAL* X, const REAL* Wt, const REAL* dY, REAL* dW, REAL* db, REAL* dX,
                int B, int in, int out_j)
{
#pragma omp parallel for schedule(static)
    for (int o = 0; o < out_j; ++o) {
        REAL sb = (REAL)0;
        for (int g = 0; g < B; ++g) sb += dY[(size_t)g * out_j + o];
        db[o] = sb;
        for (int i = 0; i < in; ++i) {
            REAL acc = (REAL)0;
            for (int g = 0; g < B; ++g) acc += dY[(size_t)g * out_j + o] * X[(size_t)g * in + i];
            dW[(size_t)o * in + i] = acc;
        }
    }
#pragma omp parallel for collapse(2) schedule(static)
    for (int g = 0; g < B; ++g)
        for (int i = 0; i < in; ++i) {
            REAL acc = (REAL)0;
            for (int o = 0; o < out_j; ++o) acc += dY[(size_t)g * out_j + o] * Wt[(size_t)o * in + i];
            dX[(size_t)g * in + i] = acc;
        }
}

/* Row losses l_g = logsumexp(Z_g) - Z[g,y_g] and dZ[g,c] = (softmax(Z_g)[c] - [c==y_g]) * scale. */
void orc_softmax_xent(const REAL* Z, const int32_t* labels, REAL* row_loss, REAL* dZ,
                      int B, int C, REAL scale)
{
    for (int g = 0; g < B; ++g) {
        const REAL* z = Z + (size_t)g * C;
        REAL m = z[0];
        for (int c = 1; c < C; ++c) if (z[c] > m) m = z[c];
        REAL s = (REAL)0;
        for (int c = 0; c < C; ++c) s += (REAL)exp((double)(z[c] - m));
        REAL lse = m + (REAL)log((double)s);
        row_loss[g] = lse - z[labels[g]];
        for (int c = 0; c < C; ++c) {
            REAL p = (REAL)exp((double)(z[c] - lse));
            dZ[(size_t)g * C + c] = (p - (c == labels[g] ? (REAL)1 : (REAL)0)) * scale;
        }
    }
}

/* v <- mu*v + g ; w <- w - lr*v. */
void orc_sgd_momentum(REAL* w, REAL* v, const REAL* g, size_t n, REAL lr, REAL mu)
{
    for (size_t i = 0; i < n; ++i) {
        REAL vn = mu * v[i] + g[i];
        v[i] = vn;
        w[i] = w[i] - lr * vn;
    }
}

int orc_real_bytes(void) { return (int)sizeof(REAL); }

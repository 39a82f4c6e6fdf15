/*
 * CPU oracle for the dense 3-D convolutions of a 3-D U-Net (test infrastructure).
 *
 * This file is TEST INFRASTRUCTURE.  It is a plain, slow, fp64, direct-loop
 * statement of what each convolution pass computes, written so that it can be
 * checked against the definitions by eye.  It shares no code with the CUDA
 * library and the library never calls it.
 *
 * What the paper fixes: the network is a U-Net, an encoder of blocks followed
 * by a decoder of blocks joined by channel-concatenation skips and a softmax
 * (Sec. 2.2, Eq. 2); filter counts double per encoder block and the decoder is
 * symmetric (Sec. 3).  Back-propagation is the chain rule applied to the
 * forward functions (Sec. 2.1, text after Eq. 1), so every backward routine
 * below is the exact adjoint / derivative of the forward definition above it.
 * The paper does not state kernel sizes; the reading used here is
 * cross-correlation with zero padding, weights stored as w[tap][c_out][c_in],
 * tap = (kd*k + kh)*k + kw.
 *
 * Layout: activations are NDHWC, channel-contiguous, dense (no pitch), fp64.
 * No blocking, no im2col, no FFT/Winograd, no BLAS.  OpenMP only spreads
 * independent output elements over threads; each output element is one
 * sequential sum in the order tap-major, channel-minor.
 */
#include <stddef.h>
#include <stdint.h>

#define IDX5(n, d, h, w, c, D, H, W, C) \
    (((((size_t)(n) * (D) + (d)) * (H) + (h)) * (W) + (w)) * (size_t)(C) + (c))

static int out_dim(int in, int k, int s, int p) { return (in + 2 * p - k) / s + 1; }

/* y[n,od,oh,ow,co] = b[co] + sum_{kd,kh,kw,ci} x[n, od*s+kd-p, oh*s+kh-p, ow*s+kw-p, ci] * w[t][co][ci]
 * (terms whose input coordinate falls outside the volume are zero). */
void orc_conv3d_fwd(const double *x, const double *w, const double *b, double *y,
                    int N, int D, int H, int W, int Ci, int Co, int k, int s, int p)
{
    const int Do = out_dim(D, k, s, p), Ho = out_dim(H, k, s, p), Wo = out_dim(W, k, s, p);
#pragma omp parallel for collapse(3) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int od = 0; od < Do; ++od)
            for (int oh = 0; oh < Ho; ++oh)
                for (int ow = 0; ow < Wo; ++ow)
                    for (int co = 0; co < Co; ++co) {
                        double acc = b ? b[co] : 0.0;
                        for (int kd = 0; kd < k; ++kd) {
                            const int id = od * s + kd - p;
                            if (id < 0 || id >= D) continue;
                            for (int kh = 0; kh < k; ++kh) {
                                const int ih = oh * s + kh - p;
                                if (ih < 0 || ih >= H) continue;
                                for (int kw = 0; kw < k; ++kw) {
                                    const int iw = ow * s + kw - p;
                                    if (iw < 0 || iw >= W) continue;
                                    const int t = (kd * k + kh) * k + kw;
                                    const double *xp = x + IDX5(n, id, ih, iw, 0, D, H, W, Ci);
                                    const double *wp = w + ((size_t)t * Co + co) * Ci;
                                    for (int ci = 0; ci < Ci; ++ci) acc += xp[ci] * wp[ci];
                                }
                            }
                        }
                        y[IDX5(n, od, oh, ow, co, Do, Ho, Wo, Co)] = acc;
                    }
}

/* dx[n,id,ih,iw,ci] = sum over (tap, output voxel) pairs with od*s+kd-p == id (same for h, w)
 *                     of dy[n,od,oh,ow,co] * w[t][co][ci]           (adjoint of the above in x).
 * D,H,W are the INPUT (dx) extents. */
void orc_conv3d_dgrad(const double *dy, const double *w, double *dx,
                      int N, int D, int H, int W, int Ci, int Co, int k, int s, int p)
{
    const int Do = out_dim(D, k, s, p), Ho = out_dim(H, k, s, p), Wo = out_dim(W, k, s, p);
#pragma omp parallel for collapse(3) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int id = 0; id < D; ++id)
            for (int ih = 0; ih < H; ++ih)
                for (int iw = 0; iw < W; ++iw)
                    for (int ci = 0; ci < Ci; ++ci) {
                        double acc = 0.0;
                        for (int kd = 0; kd < k; ++kd) {
                            const int nd = id + p - kd;
                            if (nd < 0 || nd % s) continue;
                            const int od = nd / s;
                            if (od >= Do) continue;
                            for (int kh = 0; kh < k; ++kh) {
                                const int nh = ih + p - kh;
                                if (nh < 0 || nh % s) continue;
                                const int oh = nh / s;
                                if (oh >= Ho) continue;
                                for (int kw = 0; kw < k; ++kw) {
                                    const int nw = iw + p - kw;
                                    if (nw < 0 || nw % s) continue;
                                    const int ow = nw / s;
                                    if (ow >= Wo) continue;
                                    const int t = (kd * k + kh) * k + kw;
                                    const double *gp = dy + IDX5(n, od, oh, ow, 0, Do, Ho, Wo, Co);
                                    const double *wp = w + (size_t)t * Co * Ci + ci;
                                    for (int co = 0; co < Co; ++co) acc += gp[co] * wp[(size_t)co * Ci];
                                }
                            }
                        }
                        dx[IDX5(n, id, ih, iw, ci, D, H, W, Ci)] = acc;
                    }
}

/* dw[t][co][ci] = sum_{n,od,oh,ow} dy[n,od,oh,ow,co] * x[n, od*s+kd-p, oh*s+kh-p, ow*s+kw-p, ci]
 * db[co]        = sum_{n,od,oh,ow} dy[n,od,oh,ow,co]                       (db may be NULL). */
void orc_conv3d_wgrad(const double *x, const double *dy, double *dw, double *db,
                      int N, int D, int H, int W, int Ci, int Co, int k, int s, int p)
{
    const int Do = out_dim(D, k, s, p), Ho = out_dim(H, k, s, p), Wo = out_dim(W, k, s, p);
    const int T = k * k * k;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int t = 0; t < T; ++t)
        for (int co = 0; co < Co; ++co) {
            const int kd = t / (k * k), kh = (t / k) % k, kw = t % k;
            for (int ci = 0; ci < Ci; ++ci) {
                double acc = 0.0;
                for (int n = 0; n < N; ++n)
                    for (int od = 0; od < Do; ++od) {
                        const int id = od * s + kd - p;
                        if (id < 0 || id >= D) continue;
                        for (int oh = 0; oh < Ho; ++oh) {
                            const int ih = oh * s + kh - p;
                            if (ih < 0 || ih >= H) continue;
                            for (int ow = 0; ow < Wo; ++ow) {
                                const int iw = ow * s + kw - p;
                                if (iw < 0 || iw >= W) continue;
                                acc += dy[IDX5(n, od, oh, ow, co, Do, Ho, Wo, Co)] *
                                       x[IDX5(n, id, ih, iw, ci, D, H, W, Ci)];
                            }
                        }
                    }
                dw[((size_t)t * Co + co) * Ci + ci] = acc;
            }
        }
    if (db) {
        const size_t V = (size_t)N * Do * Ho * Wo;
        for (int co = 0; co < Co; ++co) {
            double acc = 0.0;
            for (size_t v = 0; v < V; ++v) acc += dy[v * Co + co];
            db[co] = acc;
        }
    }
}

/* Transposed convolution (decoder up-sampling), output extent (D-1)*s + k per axis:
 * y[n,od,oh,ow,co] = b[co] + sum over (tap a,b,c ; input voxel d,h,w) with d*s+a == od (same for h, w)
 *                    of x[n,d,h,w,ci] * w[(a*k+b)*k+c][co][ci].
 * With k == s == 2 each output voxel receives exactly one tap of one input voxel. */
void orc_convT3d_fwd(const double *x, const double *w, const double *b, double *y,
                     int N, int D, int H, int W, int Ci, int Co, int k, int s)
{
    const int Do = (D - 1) * s + k, Ho = (H - 1) * s + k, Wo = (W - 1) * s + k;
#pragma omp parallel for collapse(3) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int od = 0; od < Do; ++od)
            for (int oh = 0; oh < Ho; ++oh)
                for (int ow = 0; ow < Wo; ++ow)
                    for (int co = 0; co < Co; ++co) {
                        double acc = b ? b[co] : 0.0;
                        for (int a = 0; a < k; ++a) {
                            const int nd = od - a;
                            if (nd < 0 || nd % s || nd / s >= D) continue;
                            for (int bb = 0; bb < k; ++bb) {
                                const int nh = oh - bb;
                                if (nh < 0 || nh % s || nh / s >= H) continue;
                                for (int c = 0; c < k; ++c) {
                                    const int nw = ow - c;
                                    if (nw < 0 || nw % s || nw / s >= W) continue;
                                    const int t = (a * k + bb) * k + c;
                                    const double *xp = x + IDX5(n, nd / s, nh / s, nw / s, 0, D, H, W, Ci);
                                    const double *wp = w + ((size_t)t * Co + co) * Ci;
                                    for (int ci = 0; ci < Ci; ++ci) acc += xp[ci] * wp[ci];
                                }
                            }
                        }
                        y[IDX5(n, od, oh, ow, co, Do, Ho, Wo, Co)] = acc;
                    }
}

/* dx[n,d,h,w,ci] = sum_{a,b,c,co} dy[n, d*s+a, h*s+b, w*s+c, co] * w[t][co][ci].  D,H,W: INPUT extents. */
void orc_convT3d_dgrad(const double *dy, const double *w, double *dx,
                       int N, int D, int H, int W, int Ci, int Co, int k, int s)
{
    const int Do = (D - 1) * s + k, Ho = (H - 1) * s + k, Wo = (W - 1) * s + k;
#pragma omp parallel for collapse(3) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int d = 0; d < D; ++d)
            for (int h = 0; h < H; ++h)
                for (int ww = 0; ww < W; ++ww)
                    for (int ci = 0; ci < Ci; ++ci) {
                        double acc = 0.0;
                        for (int a = 0; a < k; ++a)
                            for (int bb = 0; bb < k; ++bb)
                                for (int c = 0; c < k; ++c) {
                                    const int t = (a * k + bb) * k + c;
                                    const double *gp = dy + IDX5(n, d * s + a, h * s + bb, ww * s + c, 0, Do, Ho, Wo, Co);
                                    const double *wp = w + (size_t)t * Co * Ci + ci;
                                    for (int co = 0; co < Co; ++co) acc += gp[co] * wp[(size_t)co * Ci];
                                }
                        dx[IDX5(n, d, h, ww, ci, D, H, W, Ci)] = acc;
                    }
}

/* dw[t][co][ci] = sum_{n,d,h,w} dy[n, d*s+a, h*s+b, w*s+c, co] * x[n,d,h,w,ci];  db[co] = sum dy[...,co]. */
void orc_convT3d_wgrad(const double *x, const double *dy, double *dw, double *db,
                       int N, int D, int H, int W, int Ci, int Co, int k, int s)
{
    const int Do = (D - 1) * s + k, Ho = (H - 1) * s + k, Wo = (W - 1) * s + k;
    const int T = k * k * k;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int t = 0; t < T; ++t)
        for (int co = 0; co < Co; ++co) {
            const int a = t / (k * k), bb = (t / k) % k, c = t % k;
            for (int ci = 0; ci < Ci; ++ci) {
                double acc = 0.0;
                for (int n = 0; n < N; ++n)
                    for (int d = 0; d < D; ++d)
                        for (int h = 0; h < H; ++h)
                            for (int ww = 0; ww < W; ++ww)
                                acc += dy[IDX5(n, d * s + a, h * s + bb, ww * s + c, co, Do, Ho, Wo, Co)] *
                                       x[IDX5(n, d, h, ww, ci, D, H, W, Ci)];
                dw[((size_t)t * Co + co) * Ci + ci] = acc;
            }
        }
    if (db) {
        const size_t V = (size_t)N * Do * Ho * Wo;
        for (int co = 0; co < Co; ++co) {
            double acc = 0.0;
            for (size_t v = 0; v < V; ++v) acc += dy[v * Co + co];
            db[co] = acc;
        }
    }
}

/* Point-evaluated forward conv: the same sum as orc_conv3d_fwd, for a list of
 * output positions only.  pts[i] = {n, od, oh, ow}; out[i*Co + co]. */
void orc_conv3d_fwd_points(const double *x, const double *w, const double *b, const int32_t *pts, int64_t npts,
                           double *out, int N, int D, int H, int W, int Ci, int Co, int k, int s, int p)
{
    (void)N;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t i = 0; i < npts; ++i) {
        const int n = pts[4 * i], od = pts[4 * i + 1], oh = pts[4 * i + 2], ow = pts[4 * i + 3];
        for (int co = 0; co < Co; ++co) {
            double acc = b ? b[co] : 0.0;
            for (int kd = 0; kd < k; ++kd) {
                const int id = od * s + kd - p;
                if (id < 0 || id >= D) continue;
                for (int kh = 0; kh < k; ++kh) {
                    const int ih = oh * s + kh - p;
                    if (ih < 0 || ih >= H) continue;
                    for (int kw = 0; kw < k; ++kw) {
                        const int iw = ow * s + kw - p;
                        if (iw < 0 || iw >= W) continue;
                        const int t = (kd * k + kh) * k + kw;
                        const double *xp = x + IDX5(n, id, ih, iw, 0, D, H, W, Ci);
                        const double *wp = w + ((size_t)t * Co + co) * Ci;
                        for (int ci = 0; ci < Ci; ++ci) acc += xp[ci] * wp[ci];
                    }
                }
            }
            out[i * Co + co] = acc;
        }
    }
}

/* Point-evaluated weight gradient: dw entries ent[i] = {t, co, ci}; same sum as orc_conv3d_wgrad. */
void orc_conv3d_wgrad_points(const double *x, const double *dy, const int32_t *ent, int64_t nent, double *out,
                             int N, int D, int H, int W, int Ci, int Co, int k, int s, int p)
{
    const int Do = out_dim(D, k, s, p), Ho = out_dim(H, k, s, p), Wo = out_dim(W, k, s, p);
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < nent; ++i) {
        const int t = ent[3 * i], co = ent[3 * i + 1], ci = ent[3 * i + 2];
        const int kd = t / (k * k), kh = (t / k) % k, kw = t % k;
        double acc = 0.0;
        for (int n = 0; n < N; ++n)
            for (int od = 0; od < Do; ++od) {
                const int id = od * s + kd - p;
                if (id < 0 || id >= D) continue;
                for (int oh = 0; oh < Ho; ++oh) {
                    const int ih = oh * s + kh - p;
                    if (ih < 0 || ih >= H) continue;
                    for (int ow = 0; ow < Wo; ++ow) {
                        const int iw = ow * s + kw - p;
                        if (iw < 0 || iw >= W) continue;
                        acc += dy[IDX5(n, od, oh, ow, co, Do, Ho, Wo, Co)] * x[IDX5(n, id, ih, iw, ci, D, H, W, Ci)];
                    }
                }
            }
        out[i] = acc;
    }
}

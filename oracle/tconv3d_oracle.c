/*
 * CPU oracle for the three-dimensional tropical convolutions (test infrastructure, NOT a
 * product path).
 *
 * Plain nested loops over the definitions of "Compound and Parallel Modes of Tropical
 * Convolutional Neural Networks":
 *   - base operators MinPlus3d / MaxPlus3d (Section 3.2): min / max over the three-dimensional
 *     window of X[position + offset, c_in] + W[offset, c_in, c_out];
 *   - the six Conv3d layers (i)-(vi) of Section 3.2: Sum, Max or Min of a base operator over c_in;
 *   - CompoundMinPlusSumConv3d2p (section "Compound tropical convolution layers"): sum over c_in of alpha * MinPlus3d + beta *
 *     MaxPlus3d of the same weight (one shared addition per tap);
 *   - ParallelMinPlusSumConv3d2p (section "Parallel tropical convolution layers"): the same with W1 in the min branch and W2 in
 *     the max branch.
 *
 * Readings (the same as for the two-dimensional oracle): zero padding takes part in min/max as
 * x = 0; output size, stride, dilation as in PyTorch's Conv3d (Section 5 says the layers follow
 * that interface), so tensors are x[N][C][D][H][W], w[K][C][T][R][S], y[N][K][OD][OH][OW]; the
 * definition is symmetric in the three spatial axes, so which one is called depth only names the
 * memory order; ties go to the lowest flattened (c, t, r, s) (strict compares in ascending
 * order); the two-branch combine is fmaf(alpha, min, acc) then fmaf(beta, max, acc) in fp32 with
 * channels ascending; one bias per output channel added last; the backward pass routes the
 * upstream gradient wholly to the winner.  In bf16 mode every tap sum is the exact sum rounded
 * once to bf16, the channel combine stays fp32 and y is rounded once at the end.
 *
 * This file shares nothing with the CUDA path nor with the two-dimensional oracle: the tests
 * pin it against that oracle (windows of unit depth) and against an independent sliding-window
 * formulation.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { O3_MAX_PLUS = 0, O3_MIN_PLUS = 1, O3_COMPOUND = 2, O3_PARALLEL = 3 };
enum { O3_CHAN_DEFAULT = 0, O3_CHAN_SUM = 1, O3_CHAN_MAX = 2, O3_CHAN_MIN = 3 };
enum { O3_F32 = 0, O3_BF16 = 1 };

typedef struct {
    int32_t N, C, D, H, W, K, T, R, S;
    int32_t stride[3], pad[3], dil[3]; /* depth, height, width */
    int32_t mode, chan, dtype;
} o3_desc;

static int extent(int in, int pad, int dil, int k, int stride)
{
    int span = in + 2 * pad - dil * (k - 1) - 1;
    return span < 0 ? 0 : span / stride + 1;
}

int o3_output_shape(const o3_desc *d, int32_t *OD, int32_t *OH, int32_t *OW)
{
    *OD = extent(d->D, d->pad[0], d->dil[0], d->T, d->stride[0]);
    *OH = extent(d->H, d->pad[1], d->dil[1], d->R, d->stride[1]);
    *OW = extent(d->W, d->pad[2], d->dil[2], d->S, d->stride[2]);
    return 0;
}

static int chan_of(const o3_desc *d)
{
    if (d->chan != O3_CHAN_DEFAULT) return d->chan;
    if (d->mode == O3_MAX_PLUS) return O3_CHAN_MAX;
    if (d->mode == O3_MIN_PLUS) return O3_CHAN_MIN;
    return O3_CHAN_SUM;
}

/* nearest bf16 (8 significant bits, ties to even) of a finite double */
static double to_bf16(double v)
{
    if (v == 0.0) return v;
    int e;
    (void)frexp(v, &e);
    int ulp = e - 8;
    if (ulp < -133) ulp = -133;
    double r = ldexp(rint(ldexp(v, -ulp)), ulp);
    if (fabs(r) >= ldexp(1.0, 128)) r = v > 0 ? INFINITY : -INFINITY;
    return r;
}

/* one tap sum: a single binary32 add, or the exact sum rounded once to bf16 */
static float tap_sum(float xv, float wv, int dtype)
{
    if (dtype == O3_F32) {
        volatile float t = xv + wv;
        return t;
    }
    if (xv != 0.0f && wv != 0.0f) {
        int ex, ew;
        (void)frexpf(xv, &ex);
        (void)frexpf(wv, &ew);
        if (ex - ew > 40) return xv; /* the double sum below would not be exact */
        if (ew - ex > 40) return wv;
    }
    return (float)to_bf16((double)xv + (double)wv);
}

typedef struct {
    float mn, mx;
    int amn, amx; /* winning taps (t*R + r)*S + s */
} o3_window;

/* MinPlus3d and MaxPlus3d of Section 3.2 for one (n, k, c, od, oh, ow) */
static o3_window window3(const o3_desc *d, const float *x, const float *wmin, const float *wmax,
                         int n, int k, int c, int od, int oh, int ow)
{
    o3_window o = { INFINITY, -INFINITY, 0, 0 };
    for (int t = 0; t < d->T; ++t)
        for (int r = 0; r < d->R; ++r)
            for (int s = 0; s < d->S; ++s) {
                int tap = (t * d->R + r) * d->S + s;
                int id = od * d->stride[0] - d->pad[0] + t * d->dil[0];
                int ih = oh * d->stride[1] - d->pad[1] + r * d->dil[1];
                int iw = ow * d->stride[2] - d->pad[2] + s * d->dil[2];
                float xv = 0.0f;
                if (id >= 0 && id < d->D && ih >= 0 && ih < d->H && iw >= 0 && iw < d->W)
                    xv = x[((((size_t)n * d->C + c) * d->D + id) * d->H + ih) * d->W + iw];
                size_t wi = ((size_t)k * d->C + c) * d->T * d->R * d->S + tap;
                float tmn = tap_sum(xv, wmin[wi], d->dtype);
                float tmx = (wmax == wmin) ? tmn : tap_sum(xv, wmax[wi], d->dtype);
                if (tmn < o.mn) { o.mn = tmn; o.amn = tap; }
                if (tmx > o.mx) { o.mx = tmx; o.amx = tap; }
            }
    return o;
}

/*
 * Forward.  y float [N][K][OD][OH][OW].  idx (may be NULL): int32 per output, c*T*R*S + tap,
 * Max / Min channel combine.  codes (may be NULL): uint16 [N][K][C][OD][OH][OW], argmin tap in
 * the low byte, argmax tap in the high byte (T*R*S <= 256), Sum channel combine; a single-branch
 * layer fills only its own byte.  Returns 0, -1 on an invalid descriptor.
 */
int o3_forward(const o3_desc *d, const float *x, const float *w, const float *w2,
               const float *alpha, const float *beta, const float *bias, float *y, int32_t *idx,
               uint16_t *codes)
{
    int chan = chan_of(d);
    int two = (d->mode == O3_COMPOUND || d->mode == O3_PARALLEL);
    int taps = d->T * d->R * d->S;
    if (two && chan != O3_CHAN_SUM) return -1;
    if (d->mode == O3_PARALLEL && !w2) return -1;
    if (codes && taps > 256) return -1;
    int32_t OD, OH, OW;
    o3_output_shape(d, &OD, &OH, &OW);
    const float *wmax = (d->mode == O3_PARALLEL) ? w2 : w;
    size_t vol = (size_t)OD * OH * OW;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < d->N; ++n)
        for (int k = 0; k < d->K; ++k)
            for (int od = 0; od < OD; ++od)
                for (int oh = 0; oh < OH; ++oh)
                    for (int ow = 0; ow < OW; ++ow) {
                        size_t pos = ((size_t)od * OH + oh) * OW + ow;
                        float best = (chan == O3_CHAN_MAX) ? -INFINITY : INFINITY;
                        float acc = 0.0f;
                        int32_t win = -1;
                        for (int c = 0; c < d->C; ++c) {
                            o3_window o = window3(d, x, w, wmax, n, k, c, od, oh, ow);
                            size_t ci = (((size_t)n * d->K + k) * d->C + c) * vol + pos;
                            if (two) {
                                float a = alpha ? alpha[(size_t)k * d->C + c] : 1.0f;
                                float b = beta ? beta[(size_t)k * d->C + c] : 1.0f;
                                acc = fmaf(a, o.mn, acc);
                                acc = fmaf(b, o.mx, acc);
                                if (codes) codes[ci] = (uint16_t)(o.amn | (o.amx << 8));
                            } else {
                                int is_min = (d->mode == O3_MIN_PLUS);
                                float m = is_min ? o.mn : o.mx;
                                int am = is_min ? o.amn : o.amx;
                                if (chan == O3_CHAN_SUM) {
                                    volatile float sum = acc + m;
                                    acc = sum;
                                    if (codes) codes[ci] = (uint16_t)(is_min ? am : (am << 8));
                                } else if (chan == O3_CHAN_MAX) {
                                    if (m > best) { best = m; win = c * taps + am; }
                                } else {
                                    if (m < best) { best = m; win = c * taps + am; }
                                }
                            }
                        }
                        float out = (chan == O3_CHAN_SUM) ? acc : best;
                        if (bias) {
                            volatile float withb = out + bias[k];
                            out = withb;
                        }
                        if (d->dtype == O3_BF16) out = (float)to_bf16((double)out);
                        size_t oi = ((size_t)n * d->K + k) * vol + pos;
                        y[oi] = out;
                        if (idx && chan != O3_CHAN_SUM) idx[oi] = win;
                    }
    return 0;
}

/* adds v (and |v|) at index i of a gradient array and its twin of absolute sums */
static void put(double *G, double *A, size_t i, double v)
{
    if (G) G[i] += v;
    if (A) A[i] += fabs(v);
}

/*
 * Backward: the upstream gradient g[N][K][OD][OH][OW] goes wholly to the winner(s) the forward
 * rule selects (recomputed here).  All sums in double, serial, in the order (n, k, od, oh, ow, c);
 * beside each gradient G the array G_abs receives the sum of |contribution|.  Any pointer may be
 * NULL.  gx[N][C][D][H][W], gw / gw2 [K][C][T][R][S] (gw2: max branch of parallel mode),
 * galpha / gbeta [K][C], gbias [K].  Arrays are zeroed here.
 */
int o3_backward(const o3_desc *d, const float *x, const float *w, const float *w2,
                const float *alpha, const float *beta, const float *g, double *gx, double *gx_abs,
                double *gw, double *gw_abs, double *gw2, double *gw2_abs, double *galpha,
                double *galpha_abs, double *gbeta, double *gbeta_abs, double *gbias,
                double *gbias_abs)
{
    int chan = chan_of(d);
    int two = (d->mode == O3_COMPOUND || d->mode == O3_PARALLEL);
    int taps = d->T * d->R * d->S;
    if (two && chan != O3_CHAN_SUM) return -1;
    if (d->mode == O3_PARALLEL && !w2) return -1;
    int32_t OD, OH, OW;
    o3_output_shape(d, &OD, &OH, &OW);
    const float *wmax = (d->mode == O3_PARALLEL) ? w2 : w;
    size_t nx = (size_t)d->N * d->C * d->D * d->H * d->W, nw = (size_t)d->K * d->C * taps;
    size_t nab = (size_t)d->K * d->C, nb = (size_t)d->K;
    double *arrs[12] = { gx, gx_abs, gw, gw_abs, gw2, gw2_abs, galpha, galpha_abs, gbeta, gbeta_abs,
                         gbias, gbias_abs };
    size_t lens[12] = { nx, nx, nw, nw, nw, nw, nab, nab, nab, nab, nb, nb };
    for (int a = 0; a < 12; ++a)
        if (arrs[a]) memset(arrs[a], 0, lens[a] * sizeof(double));
    size_t vol = (size_t)OD * OH * OW;
    for (int n = 0; n < d->N; ++n)
        for (int k = 0; k < d->K; ++k)
            for (int od = 0; od < OD; ++od)
                for (int oh = 0; oh < OH; ++oh)
                    for (int ow = 0; ow < OW; ++ow) {
                        double gv = g[((size_t)n * d->K + k) * vol + ((size_t)od * OH + oh) * OW + ow];
                        put(gbias, gbias_abs, k, gv);
                        float best = (chan == O3_CHAN_MAX) ? -INFINITY : INFINITY;
                        int best_c = -1, best_tap = 0;
                        for (int c = 0; c < d->C; ++c) {
                            o3_window o = window3(d, x, w, wmax, n, k, c, od, oh, ow);
                            if (chan != O3_CHAN_SUM) {
                                float m = (d->mode == O3_MIN_PLUS) ? o.mn : o.mx;
                                int am = (d->mode == O3_MIN_PLUS) ? o.amn : o.amx;
                                int better = (chan == O3_CHAN_MAX) ? (m > best) : (m < best);
                                if (better) { best = m; best_c = c; best_tap = am; }
                                continue;
                            }
                            for (int br = 0; br < 2; ++br) { /* 0: min branch, 1: max branch */
                                if (!two && (br == 0) != (d->mode == O3_MIN_PLUS)) continue;
                                int tap = br == 0 ? o.amn : o.amx;
                                double coef = 1.0;
                                if (two) {
                                    const float *ab = br == 0 ? alpha : beta;
                                    coef = ab ? (double)ab[(size_t)k * d->C + c] : 1.0;
                                }
                                size_t wi = ((size_t)k * d->C + c) * taps + tap;
                                if (d->mode == O3_PARALLEL && br == 1) put(gw2, gw2_abs, wi, coef * gv);
                                else put(gw, gw_abs, wi, coef * gv);
                                int t = tap / (d->R * d->S), r = (tap / d->S) % d->R, s = tap % d->S;
                                int id = od * d->stride[0] - d->pad[0] + t * d->dil[0];
                                int ih = oh * d->stride[1] - d->pad[1] + r * d->dil[1];
                                int iw = ow * d->stride[2] - d->pad[2] + s * d->dil[2];
                                if (id >= 0 && id < d->D && ih >= 0 && ih < d->H && iw >= 0 && iw < d->W)
                                    put(gx, gx_abs,
                                        ((((size_t)n * d->C + c) * d->D + id) * d->H + ih) * d->W + iw,
                                        coef * gv);
                                if (two) {
                                    double val = br == 0 ? (double)o.mn : (double)o.mx;
                                    if (br == 0) put(galpha, galpha_abs, (size_t)k * d->C + c, gv * val);
                                    else put(gbeta, gbeta_abs, (size_t)k * d->C + c, gv * val);
                                }
                            }
                        }
                        if (chan != O3_CHAN_SUM && best_c >= 0) {
                            put(gw, gw_abs, ((size_t)k * d->C + best_c) * taps + best_tap, gv);
                            int t = best_tap / (d->R * d->S), r = (best_tap / d->S) % d->R,
                                s = best_tap % d->S;
                            int id = od * d->stride[0] - d->pad[0] + t * d->dil[0];
                            int ih = oh * d->stride[1] - d->pad[1] + r * d->dil[1];
                            int iw = ow * d->stride[2] - d->pad[2] + s * d->dil[2];
                            if (id >= 0 && id < d->D && ih >= 0 && ih < d->H && iw >= 0 && iw < d->W)
                                put(gx, gx_abs,
                                    ((((size_t)n * d->C + best_c) * d->D + id) * d->H + ih) * d->W + iw, gv);
                        }
                    }
    return 0;
}

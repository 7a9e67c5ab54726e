/*
 * CPU oracle for tropical convolution (test infrastructure, NOT a product path).
 *
 * Plain nested loops that write out the definitions of the paper
 * "Compound and Parallel Modes of Tropical Convolutional Neural Networks":
 *   - base operators MinPlus2d / MaxPlus2d (Section 3.1): min / max over the
 *     Kh x Kw window of X[h+i, w+j, c_in] + W[i, j, c_in, c_out];
 *   - the six TCNN layers (i)-(vi) of Section 3.1: Sum, Max or Min of the base
 *     operator over c_in;
 *   - the compound layer (section "Compound tropical convolution layers",
 *     CompoundMinPlusSumConv2d2p):
 *       Y = sum_c ( alpha[c,k] * MinPlus2d(X,W) + beta[c,k] * MaxPlus2d(X,W) ),
 *     where both branches share the same addition (remark closing that section);
 *   - the parallel layer (section "Parallel tropical convolution layers",
 *     ParallelMinPlusSumConv2d2p): the same
 *     with W1 in the min branch and W2 in the max branch;
 *   - the operation counts of Section 4.1 (instrumented counters).
 *
 * Readings where the paper is silent (each is stated in the repository's
 * design notes): zero padding takes part in min/max as x = 0; output size,
 * stride and dilation follow the PyTorch convolution convention the paper says
 * its layers follow (Section 5); ties go to the lowest flattened (c, r, s)
 * (strict compares in ascending order); one bias per output channel added
 * last; alpha/beta stored [K][C]; the backward pass routes the upstream
 * gradient wholly to the winner.  Parity unpinned by the paper: padding value,
 * gradient tie rule, alpha/beta memory layout, bias placement.
 *
 * Second padding reading (pad_mode = 1, "neutral"): a padded tap holds the
 * identity of the branch's semiring (+inf for min-plus, -inf for max-plus; the
 * section "Tropical algebra and tropical convolution" gives these identities),
 * i.e. it never takes part in the min / max: the tap is skipped.  A window that
 * lies wholly in the padding yields the identity itself.
 *
 * Tensors are dense: x[N][C][H][W], w/w2[K][C][R][S], y/g[N][K][OH][OW],
 * alpha/beta[K][C], bias[K].  All values travel as float; in bf16 mode the
 * caller guarantees they are bf16-representable and every tap sum is rounded
 * once (round-to-nearest-even) to bf16, the channel combine stays fp32 and y is
 * rounded to bf16 at the end.
 *
 * This file shares nothing with the CUDA path: no header, no helper, no table.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORA_MAX_PLUS = 0, ORA_MIN_PLUS = 1, ORA_COMPOUND = 2, ORA_PARALLEL = 3 };
enum { ORA_CHAN_DEFAULT = 0, ORA_CHAN_SUM = 1, ORA_CHAN_MAX = 2, ORA_CHAN_MIN = 3 };
enum { ORA_F32 = 0, ORA_BF16 = 1 };

typedef struct {
    int32_t N, C, H, W, K, R, S;
    int32_t stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
    int32_t mode, chan, dtype;
    int32_t pad_mode; /* 0: zero padding takes part as x = 0; 1: padded taps are skipped */
} ora_desc;

/* Section 4.1 tallies: additions, comparisons, multiplications. */
typedef struct {
    int64_t adds, cmps, muls;
} ora_counts;

static int out_extent(int in, int pad, int dil, int k, int stride)
{
    /* PyTorch convolution arithmetic (the convention Section 5 adopts). */
    int span = in + 2 * pad - dil * (k - 1) - 1;
    if (span < 0) return 0;
    return span / stride + 1;
}

int ora_output_shape(const ora_desc *d, int32_t *OH, int32_t *OW)
{
    *OH = out_extent(d->H, d->pad_h, d->dil_h, d->R, d->stride_h);
    *OW = out_extent(d->W, d->pad_w, d->dil_w, d->S, d->stride_w);
    return 0;
}

static int resolved_chan(const ora_desc *d)
{
    if (d->chan != ORA_CHAN_DEFAULT) return d->chan;
    if (d->mode == ORA_MAX_PLUS) return ORA_CHAN_MAX; /* layer (v)  */
    if (d->mode == ORA_MIN_PLUS) return ORA_CHAN_MIN; /* layer (iv) */
    return ORA_CHAN_SUM;                              /* compound / parallel */
}

int ora_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Round a double to the nearest bf16 value (8 significant bits, exponent range
 * of binary32, ties to even).  v is assumed finite. */
static double round_to_bf16(double v)
{
    if (v == 0.0) return v;
    int e;
    (void)frexp(v, &e);            /* |v| = m * 2^e, m in [0.5, 1) */
    int ulp_exp = e - 8;           /* 8 significant bits */
    if (ulp_exp < -133) ulp_exp = -133; /* bf16 subnormal spacing 2^-133 */
    double q = rint(ldexp(v, -ulp_exp)); /* default rounding mode: nearest even */
    double r = ldexp(q, ulp_exp);
    if (fabs(r) >= ldexp(1.0, 128)) r = (v > 0) ? INFINITY : -INFINITY;
    return r;
}

/* One tap sum in the layer's arithmetic type.  fp32: one IEEE binary32 add.
 * bf16: the exact sum rounded once to bf16.  (Two bf16 values whose exponents
 * differ by more than 40 binary orders sum, after rounding, to the larger one;
 * otherwise the double sum is exact.) */
static float tap_add(float xv, float wv, int dtype)
{
    if (dtype == ORA_F32) {
        volatile float t = xv + wv; /* volatile: no extended precision, no contraction */
        return t;
    }
    if (xv != 0.0f && wv != 0.0f) {
        int ex, ew;
        (void)frexpf(xv, &ex);
        (void)frexpf(wv, &ew);
        if (ex - ew > 40) return xv;
        if (ew - ex > 40) return wv;
    }
    return (float)round_to_bf16((double)xv + (double)wv);
}

typedef struct {
    float mn, mx; /* MinPlus2d, MaxPlus2d of this (n, k, c, oh, ow) */
    int amn, amx; /* their winning taps r*S+s (lowest tap on ties)  */
} ora_window;

/* Base operators of Section 3.1 for one (n, k, c, oh, ow).  wmin feeds the min
 * branch, wmax the max branch (the same array except in parallel mode).  When
 * they are the same array the tap sum is computed once and shared. */
static ora_window base_ops(const ora_desc *d, const float *x, const float *wmin,
                           const float *wmax, int n, int k, int c, int oh, int ow,
                           ora_counts *cnt, int want_min, int want_max)
{
    ora_window o;
    o.mn = INFINITY;
    o.mx = -INFINITY;
    o.amn = 0;
    o.amx = 0;
    for (int r = 0; r < d->R; ++r) {
        for (int s = 0; s < d->S; ++s) {
            int tap = r * d->S + s;
            int ih = oh * d->stride_h - d->pad_h + r * d->dil_h;
            int iw = ow * d->stride_w - d->pad_w + s * d->dil_w;
            float xv = 0.0f; /* zero padding */
            if (ih >= 0 && ih < d->H && iw >= 0 && iw < d->W)
                xv = x[(((size_t)n * d->C + c) * d->H + ih) * d->W + iw];
            else if (d->pad_mode == 1)
                continue; /* neutral padding: the tap holds the semiring identity */
            size_t wi = (((size_t)k * d->C + c) * d->R + r) * d->S + s;
            float tmn = tap_add(xv, wmin[wi], d->dtype);
            float tmx = tmn;
            if (cnt) cnt->adds += 1;
            if (wmax != wmin) {
                tmx = tap_add(xv, wmax[wi], d->dtype);
                if (cnt) cnt->adds += 1;
            }
            if (want_min) {
                if (cnt && tap > 0) cnt->cmps += 1;
                if (tmn < o.mn) { o.mn = tmn; o.amn = tap; }
            }
            if (want_max) {
                if (cnt && tap > 0) cnt->cmps += 1;
                if (tmx > o.mx) { o.mx = tmx; o.amx = tap; }
            }
        }
    }
    return o;
}

/*
 * Forward pass.  y[N][K][OH][OW] (float; bf16-representable in bf16 mode).
 * idx (may be NULL): int32 [N][K][OH][OW] = c*R*S + r*S + s, written for the
 *   Max / Min channel combines.
 * codes (may be NULL): uint8 [N][K][C][OH][OW], low nibble = argmin tap, high
 *   nibble = argmax tap (a single-branch Sum layer fills only its own nibble),
 *   written for the Sum channel combine; needs R*S <= 16.
 * cnt (may be NULL): Section 4.1 tallies; the run is serial when requested.
 * Returns 0, or -1 on an invalid descriptor.
 */
int ora_forward(const ora_desc *d, const float *x, const float *w, const float *w2,
                const float *alpha, const float *beta, const float *bias, float *y,
                int32_t *idx, uint8_t *codes, ora_counts *cnt)
{
    int chan = resolved_chan(d);
    int two_branch = (d->mode == ORA_COMPOUND || d->mode == ORA_PARALLEL);
    if (two_branch && chan != ORA_CHAN_SUM) return -1;
    if (d->mode == ORA_PARALLEL && !w2) return -1;
    if (codes && d->R * d->S > 16) return -1;
    int32_t OH, OW;
    ora_output_shape(d, &OH, &OW);
    const float *wmin = w;
    const float *wmax = (d->mode == ORA_PARALLEL) ? w2 : w;
    int RS = d->R * d->S;
    int want_min = two_branch || d->mode == ORA_MIN_PLUS;
    int want_max = two_branch || d->mode == ORA_MAX_PLUS;
    if (cnt) { cnt->adds = cnt->cmps = cnt->muls = 0; }

#pragma omp parallel for collapse(2) schedule(static) if (!cnt)
    for (int n = 0; n < d->N; ++n) {
        for (int k = 0; k < d->K; ++k) {
            for (int oh = 0; oh < OH; ++oh) {
                for (int ow = 0; ow < OW; ++ow) {
                    float best = (chan == ORA_CHAN_MAX) ? -INFINITY : INFINITY;
                    float acc = 0.0f;
                    int32_t win = -1;
                    for (int c = 0; c < d->C; ++c) {
                        ora_window o = base_ops(d, x, wmin, wmax, n, k, c, oh, ow, cnt,
                                                want_min, want_max);
                        if (two_branch) {
                            /* compound / parallel layer definitions: alpha * MinPlus2d + beta * MaxPlus2d,
                             * min branch first, each a fused multiply-add in fp32 */
                            float a = alpha ? alpha[(size_t)k * d->C + c] : 1.0f;
                            float b = beta ? beta[(size_t)k * d->C + c] : 1.0f;
                            acc = fmaf(a, o.mn, acc);
                            acc = fmaf(b, o.mx, acc);
                            if (cnt) { cnt->muls += 2; cnt->adds += (c == 0) ? 1 : 2; }
                            if (codes)
                                codes[((((size_t)n * d->K + k) * d->C + c) * OH + oh) * OW + ow] =
                                    (uint8_t)(o.amn | (o.amx << 4));
                        } else {
                            float m = (d->mode == ORA_MIN_PLUS) ? o.mn : o.mx;
                            int am = (d->mode == ORA_MIN_PLUS) ? o.amn : o.amx;
                            if (chan == ORA_CHAN_SUM) {
                                volatile float sum = acc + m; /* layers (i), (ii) */
                                acc = sum;
                                if (cnt && c > 0) cnt->adds += 1;
                                if (codes)
                                    codes[((((size_t)n * d->K + k) * d->C + c) * OH + oh) * OW + ow] =
                                        (uint8_t)((d->mode == ORA_MIN_PLUS) ? am : (am << 4));
                            } else if (chan == ORA_CHAN_MAX) { /* layers (iii), (v) */
                                if (cnt && c > 0) cnt->cmps += 1;
                                if (m > best) { best = m; win = c * RS + am; }
                            } else { /* layers (iv), (vi) */
                                if (cnt && c > 0) cnt->cmps += 1;
                                if (m < best) { best = m; win = c * RS + am; }
                            }
                        }
                    }
                    float out = (chan == ORA_CHAN_SUM) ? acc : best;
                    if (bias) {
                        volatile float withb = out + bias[k];
                        out = withb;
                    }
                    if (d->dtype == ORA_BF16) out = (float)round_to_bf16((double)out);
                    size_t oi = (((size_t)n * d->K + k) * OH + oh) * OW + ow;
                    y[oi] = out;
                    if (idx && chan != ORA_CHAN_SUM) idx[oi] = win;
                }
            }
        }
    }
    return 0;
}

/*
 * Backward pass: the upstream gradient g[N][K][OH][OW] is routed wholly to the
 * winner(s) the forward rule selects (recomputed here).  Every sum is
 * accumulated in double; beside each gradient array G the array G_abs receives
 * the sum of |contribution| (the scale of the summation error bound).  Any
 * output pointer may be NULL.  Sizes: gx[N][C][H][W], gw/gw2[K][C][R][S],
 * galpha/gbeta[K][C], gbias[K].  gw2 is used by parallel mode only (max branch).
 */
int ora_backward(const ora_desc *d, const float *x, const float *w, const float *w2,
                 const float *alpha, const float *beta, const float *g,
                 double *gx, double *gx_abs, double *gw, double *gw_abs,
                 double *gw2, double *gw2_abs, double *galpha, double *galpha_abs,
                 double *gbeta, double *gbeta_abs, double *gbias, double *gbias_abs)
{
    int chan = resolved_chan(d);
    int two_branch = (d->mode == ORA_COMPOUND || d->mode == ORA_PARALLEL);
    if (two_branch && chan != ORA_CHAN_SUM) return -1;
    if (d->mode == ORA_PARALLEL && !w2) return -1;
    int32_t OH, OW;
    ora_output_shape(d, &OH, &OW);
    const float *wmin = w;
    const float *wmax = (d->mode == ORA_PARALLEL) ? w2 : w;
    int want_min = two_branch || d->mode == ORA_MIN_PLUS;
    int want_max = two_branch || d->mode == ORA_MAX_PLUS;
    size_t nx = (size_t)d->N * d->C * d->H * d->W;
    size_t nw = (size_t)d->K * d->C * d->R * d->S;
    size_t nab = (size_t)d->K * d->C;
    size_t nb = (size_t)d->K;
    /* parameter gradients: one private set per thread, merged in thread order */
    int T = ora_threads();
    size_t per = 2 * nw * 2 + 2 * nab * 2 + 2 * nb; /* gw,gw2,ga,gb,gbias with abs twins */
    double *priv = (double *)calloc((size_t)T * per, sizeof(double));
    if (!priv) return -2;
    if (gx) memset(gx, 0, nx * sizeof(double));
    if (gx_abs) memset(gx_abs, 0, nx * sizeof(double));

#pragma omp parallel for schedule(static) num_threads(T)
    for (int n = 0; n < d->N; ++n) {
#ifdef _OPENMP
        int tid = omp_get_thread_num();
#else
        int tid = 0;
#endif
        double *p = priv + (size_t)tid * per;
        double *Pgw = p, *Pgw_abs = Pgw + nw, *Pgw2 = Pgw_abs + nw, *Pgw2_abs = Pgw2 + nw;
        double *Pga = Pgw2_abs + nw, *Pga_abs = Pga + nab, *Pgb = Pga_abs + nab,
               *Pgb_abs = Pgb + nab;
        double *Pbias = Pgb_abs + nab, *Pbias_abs = Pbias + nb;
        for (int k = 0; k < d->K; ++k) {
            for (int oh = 0; oh < OH; ++oh) {
                for (int ow = 0; ow < OW; ++ow) {
                    double gv = (double)g[(((size_t)n * d->K + k) * OH + oh) * OW + ow];
                    Pbias[k] += gv;
                    Pbias_abs[k] += fabs(gv);
                    /* winner search exactly as in the forward pass */
                    float best = (chan == ORA_CHAN_MAX) ? -INFINITY : INFINITY;
                    int best_c = -1, best_tap = 0;
                    for (int c = 0; c < d->C; ++c) {
                        ora_window o = base_ops(d, x, wmin, wmax, n, k, c, oh, ow, NULL,
                                                want_min, want_max);
                        if (chan == ORA_CHAN_SUM) {
                            /* one winner per branch per (output, c) */
                            for (int br = 0; br < 2; ++br) {
                                int is_min = (br == 0);
                                if (is_min && !want_min) continue;
                                if (!is_min && !want_max) continue;
                                int tap = is_min ? o.amn : o.amx;
                                double coef = 1.0;
                                if (two_branch) {
                                    const float *ab = is_min ? alpha : beta;
                                    coef = ab ? (double)ab[(size_t)k * d->C + c] : 1.0;
                                }
                                double contrib = coef * gv;
                                int r = tap / d->S, s = tap % d->S;
                                size_t wi = (((size_t)k * d->C + c) * d->R + r) * d->S + s;
                                if (d->mode == ORA_PARALLEL && !is_min) {
                                    Pgw2[wi] += contrib;
                                    Pgw2_abs[wi] += fabs(contrib);
                                } else {
                                    Pgw[wi] += contrib;
                                    Pgw_abs[wi] += fabs(contrib);
                                }
                                int ih = oh * d->stride_h - d->pad_h + r * d->dil_h;
                                int iw = ow * d->stride_w - d->pad_w + s * d->dil_w;
                                if (ih >= 0 && ih < d->H && iw >= 0 && iw < d->W) {
                                    size_t xi = (((size_t)n * d->C + c) * d->H + ih) * d->W + iw;
                                    if (gx) gx[xi] += contrib;
                                    if (gx_abs) gx_abs[xi] += fabs(contrib);
                                }
                                if (two_branch) {
                                    double val = is_min ? (double)o.mn : (double)o.mx;
                                    double *G = is_min ? Pga : Pgb;
                                    double *A = is_min ? Pga_abs : Pgb_abs;
                                    G[(size_t)k * d->C + c] += gv * val;
                                    A[(size_t)k * d->C + c] += fabs(gv * val);
                                }
                            }
                        } else {
                            float m = (d->mode == ORA_MIN_PLUS) ? o.mn : o.mx;
                            int am = (d->mode == ORA_MIN_PLUS) ? o.amn : o.amx;
                            int better = (chan == ORA_CHAN_MAX) ? (m > best) : (m < best);
                            if (better) { best = m; best_c = c; best_tap = am; }
                        }
                    }
                    if (chan != ORA_CHAN_SUM && best_c >= 0) {
                        int r = best_tap / d->S, s = best_tap % d->S;
                        size_t wi = (((size_t)k * d->C + best_c) * d->R + r) * d->S + s;
                        Pgw[wi] += gv;
                        Pgw_abs[wi] += fabs(gv);
                        int ih = oh * d->stride_h - d->pad_h + r * d->dil_h;
                        int iw = ow * d->stride_w - d->pad_w + s * d->dil_w;
                        if (ih >= 0 && ih < d->H && iw >= 0 && iw < d->W) {
                            size_t xi = (((size_t)n * d->C + best_c) * d->H + ih) * d->W + iw;
                            if (gx) gx[xi] += gv;
                            if (gx_abs) gx_abs[xi] += fabs(gv);
                        }
                    }
                }
            }
        }
    }

    /* merge the per-thread parameter gradients in thread order */
    double *outs[10] = { gw, gw_abs, gw2, gw2_abs, galpha, galpha_abs, gbeta, gbeta_abs,
                         gbias, gbias_abs };
    size_t lens[10] = { nw, nw, nw, nw, nab, nab, nab, nab, nb, nb };
    size_t off = 0;
    for (int a = 0; a < 10; ++a) {
        if (outs[a]) {
            for (size_t i = 0; i < lens[a]; ++i) {
                double sacc = 0.0;
                for (int t = 0; t < T; ++t) sacc += priv[(size_t)t * per + off + i];
                outs[a][i] = sacc;
            }
        }
        off += lens[a];
    }
    free(priv);
    return 0;
}

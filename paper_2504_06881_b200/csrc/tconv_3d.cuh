// Three-dimensional tropical convolution (Section 3.2 and the Conv3d forms of Sections 3.4, 3.5).
// The paper's 3-D workloads are LeNet-sized (one to sixteen channels, 5 x 5 x 5 windows on 28^3 and
// 64^3 volumes): a window has many taps and few channels, so one thread owns one output position
// for a few output channels, the weights of a channel chunk sit in shared memory and the input is
// read through L1 (neighbouring threads read neighbouring elements).  All kernels are
// deterministic and atomic-free.
#pragma once
#include "tconv_common.cuh"

namespace tconv {

struct Geo3 {
    int N, C, D, H, W, K, T, R, S;
    int sd, sh, sw, pd, ph, pw, dd, dh, dw;
    int OD, OH, OW, taps, vol;  // vol = OD*OH*OW
    int mode, chan;
};

constexpr int kFwd3Threads = 128;

// Forward.  grid (ceil(N * vol / 128), ceil(K / KT)): one thread per (n, output position) of the
// flattened range, KT output channels each.  Shared memory: weights of `cch` input channels for
// this block's KT output channels, [cc][tap][KT] (twice in parallel mode), as T.
// WIN: track the winning taps (strict compares, taps ascending); without it the extrema are plain
// min / max.  SC: the window's innermost extent S when it is 3 or 5 (unrolled), else 0.
template <typename T, int KT, bool WIN, int SC>
__global__ void __launch_bounds__(kFwd3Threads)
fwd3d_kernel(Geo3 g, int cch, const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ w2,
             const float* __restrict__ alpha, const float* __restrict__ beta,
             const float* __restrict__ bias, T* __restrict__ y, void* __restrict__ winners) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    T* wmin_s = reinterpret_cast<T*>(smem_raw);
    const bool par = g.mode == TCONV_PARALLEL;
    const bool twob = two_branch(g.mode);
    T* wmax_s = par ? wmin_s + (size_t)cch * g.taps * KT : wmin_s;
    const long long flat = (long long)blockIdx.x * kFwd3Threads + threadIdx.x;
    const bool live = flat < (long long)g.N * g.vol;
    const int n = live ? (int)(flat / g.vol) : 0, pos = live ? (int)(flat % g.vol) : 0;
    const int k0 = blockIdx.y * KT;
    const int ow = pos % g.OW, oh = (pos / g.OW) % g.OH, od = pos / (g.OW * g.OH);
    const int d0 = od * g.sd - g.pd, h0 = oh * g.sh - g.ph, w0 = ow * g.sw - g.pw;
    const int S = SC ? SC : g.S;
    float acc[KT], best[KT];
    int win[KT];
#pragma unroll
    for (int j = 0; j < KT; ++j) {
        acc[j] = 0.0f;
        best[j] = (g.chan == CH_MAX) ? -INFINITY : INFINITY;
        win[j] = -1;
    }
    for (int c0 = 0; c0 < g.C; c0 += cch) {
        const int ncc = min(cch, g.C - c0);
        __syncthreads();
        for (int i = threadIdx.x; i < ncc * g.taps * KT; i += kFwd3Threads) {
            const int j = i % KT, tap = (i / KT) % g.taps, cc = i / (KT * g.taps);
            const int k = k0 + j;
            const size_t wi = ((size_t)k * g.C + c0 + cc) * g.taps + tap;
            wmin_s[i] = k < g.K ? w[wi] : zero_of<T>();
            if (par) wmax_s[i] = k < g.K ? w2[wi] : zero_of<T>();
        }
        __syncthreads();
        if (!live) continue;
        for (int cc = 0; cc < ncc; ++cc) {
            const int c = c0 + cc;
            const T* xc = x + ((size_t)n * g.C + c) * g.D * g.H * g.W;
            const T* wa = wmin_s + (size_t)cc * g.taps * KT;
            const T* wb = wmax_s + (size_t)cc * g.taps * KT;
            float mn[KT], mx[KT];
            int amn[KT], amx[KT];
#pragma unroll
            for (int j = 0; j < KT; ++j) {
                mn[j] = INFINITY; mx[j] = -INFINITY; amn[j] = 0; amx[j] = 0;
            }
            int tap = 0;
            for (int t = 0; t < g.T; ++t) {
                const int id = d0 + t * g.dd;
                const bool okd = id >= 0 && id < g.D;
                for (int r = 0; r < g.R; ++r) {
                    const int ih = h0 + r * g.dh;
                    const bool okh = okd && ih >= 0 && ih < g.H;
                    const T* xrow = xc + ((size_t)(okh ? id : 0) * g.H + (okh ? ih : 0)) * g.W;
                    if constexpr (SC != 0) {
                        T xv[SC];
#pragma unroll
                        for (int s = 0; s < SC; ++s) {
                            const int iw = w0 + s * g.dw;
                            xv[s] = (okh && iw >= 0 && iw < g.W) ? xrow[iw] : zero_of<T>();
                        }
#pragma unroll
                        for (int s = 0; s < SC; ++s) {
#pragma unroll
                            for (int j = 0; j < KT; ++j) {
                                const float tmn = tap_add(xv[s], wa[(tap + s) * KT + j]);
                                const float tmx = par ? tap_add(xv[s], wb[(tap + s) * KT + j]) : tmn;
                                if constexpr (WIN) {
                                    if (tmn < mn[j]) { mn[j] = tmn; amn[j] = tap + s; }
                                    if (tmx > mx[j]) { mx[j] = tmx; amx[j] = tap + s; }
                                } else {
                                    mn[j] = fminf(mn[j], tmn);
                                    mx[j] = fmaxf(mx[j], tmx);
                                }
                            }
                        }
                        tap += SC;
                    } else {
                        for (int s = 0; s < S; ++s, ++tap) {
                            const int iw = w0 + s * g.dw;
                            T xv = zero_of<T>();
                            if (okh && iw >= 0 && iw < g.W) xv = xrow[iw];
#pragma unroll
                            for (int j = 0; j < KT; ++j) {
                                const float tmn = tap_add(xv, wa[tap * KT + j]);
                                const float tmx = par ? tap_add(xv, wb[tap * KT + j]) : tmn;
                                if constexpr (WIN) {
                                    if (tmn < mn[j]) { mn[j] = tmn; amn[j] = tap; }
                                    if (tmx > mx[j]) { mx[j] = tmx; amx[j] = tap; }
                                } else {
                                    mn[j] = fminf(mn[j], tmn);
                                    mx[j] = fmaxf(mx[j], tmx);
                                }
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < KT; ++j) {
                const int k = k0 + j;
                if (k >= g.K) continue;
                if (twob) {
                    const float a = alpha ? alpha[(size_t)k * g.C + c] : 1.0f;
                    const float b = beta ? beta[(size_t)k * g.C + c] : 1.0f;
                    acc[j] = __fmaf_rn(a, mn[j], acc[j]);
                    acc[j] = __fmaf_rn(b, mx[j], acc[j]);
                } else {
                    const bool is_min = g.mode == TCONV_MIN_PLUS;
                    const float m = is_min ? mn[j] : mx[j];
                    const int am = is_min ? amn[j] : amx[j];
                    if (g.chan == CH_SUM) acc[j] = __fadd_rn(acc[j], m);
                    else if (g.chan == CH_MAX) { if (m > best[j]) { best[j] = m; win[j] = c * g.taps + am; } }
                    else { if (m < best[j]) { best[j] = m; win[j] = c * g.taps + am; } }
                    if (is_min) amx[j] = 0; else amn[j] = 0;
                }
                if (WIN && g.chan == CH_SUM)
                    ((uint16_t*)winners)[(((size_t)n * g.K + k) * g.C + c) * g.vol + pos] =
                        (uint16_t)(amn[j] | (amx[j] << 8));
            }
        }
    }
    if (!live) return;
#pragma unroll
    for (int j = 0; j < KT; ++j) {
        const int k = k0 + j;
        if (k >= g.K) continue;
        float out = (g.chan == CH_SUM) ? acc[j] : best[j];
        if (bias) out = __fadd_rn(out, bias[k]);
        const size_t o = ((size_t)n * g.K + k) * g.vol + pos;
        if (y) y[o] = from_f32<T>(out);
        if (WIN && g.chan != CH_SUM) ((int32_t*)winners)[o] = win[j];
    }
}

// The winning taps of (n, k, c, position) as two ints; -1 where the layer has no such branch or
// (Max / Min channel combine) another channel won.
__device__ __forceinline__ void winners3(const Geo3& g, const void* winners, int n, int k, int c, int pos,
                                         int& amn, int& amx) {
    if (g.chan == CH_SUM) {
        const unsigned v = ((const uint16_t*)winners)[(((size_t)n * g.K + k) * g.C + c) * g.vol + pos];
        amn = (g.mode == TCONV_MAX_PLUS) ? -1 : (int)(v & 0xFFu);
        amx = (g.mode == TCONV_MIN_PLUS) ? -1 : (int)(v >> 8);
    } else {
        const int v = ((const int32_t*)winners)[((size_t)n * g.K + k) * g.vol + pos] - c * g.taps;
        const int tap = (v >= 0 && v < g.taps) ? v : -1;
        amn = (g.mode == TCONV_MIN_PLUS) ? tap : -1;
        amx = (g.mode == TCONV_MIN_PLUS) ? -1 : tap;
    }
}

// grad_x in gather form.  A block of 256 threads owns 256 / slices consecutive input elements
// (threadIdx.x) and splits the output channels over blockDim.y = 1, 2, 4 or 8 slices (k = slice, slice + slices, ...): each thread visits,
// taps ascending and its channels ascending inside a tap, the outputs whose window reads its
// element; the slices' partial sums are then added in slice order.  (Small 3-D layers have few
// input elements: the slices keep enough warps in flight to hide the dependent loads.)
constexpr int kGx3Slices = 8;

template <typename T>
__global__ void __launch_bounds__(32 * kGx3Slices)
bwd3d_gx_kernel(Geo3 g, const float* __restrict__ alpha, const float* __restrict__ beta,
                const T* __restrict__ gy, const void* __restrict__ winners, T* __restrict__ gx) {
    __shared__ float part[32 * kGx3Slices];
    const size_t total = (size_t)g.N * g.C * g.D * g.H * g.W;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int slice = threadIdx.y, slices = blockDim.y;
    const bool live = i < total;
    const bool twob = two_branch(g.mode);
    float acc = 0.0f;
    if (live) {
        const int iw = (int)(i % g.W), ih = (int)((i / g.W) % g.H), id = (int)((i / ((size_t)g.W * g.H)) % g.D);
        const int c = (int)((i / ((size_t)g.W * g.H * g.D)) % g.C),
                  n = (int)(i / ((size_t)g.W * g.H * g.D * g.C));
        for (int t = 0; t < g.T; ++t) {
            const int nd = id + g.pd - t * g.dd;
            if (nd < 0 || nd % g.sd != 0 || nd / g.sd >= g.OD) continue;
            for (int r = 0; r < g.R; ++r) {
                const int nh = ih + g.ph - r * g.dh;
                if (nh < 0 || nh % g.sh != 0 || nh / g.sh >= g.OH) continue;
                for (int s = 0; s < g.S; ++s) {
                    const int nw = iw + g.pw - s * g.dw;
                    if (nw < 0 || nw % g.sw != 0 || nw / g.sw >= g.OW) continue;
                    const int tap = (t * g.R + r) * g.S + s;
                    const int pos = ((nd / g.sd) * g.OH + nh / g.sh) * g.OW + nw / g.sw;
                    for (int k = slice; k < g.K; k += slices) {
                        int amn, amx;
                        winners3(g, winners, n, k, c, pos, amn, amx);
                        if (amn != tap && amx != tap) continue;
                        const float gv = to_f32(gy[((size_t)n * g.K + k) * g.vol + pos]);
                        if (twob) {
                            const float a = alpha ? alpha[(size_t)k * g.C + c] : 1.0f;
                            const float b = beta ? beta[(size_t)k * g.C + c] : 1.0f;
                            if (amn == tap) acc = __fmaf_rn(a, gv, acc);
                            if (amx == tap) acc = __fmaf_rn(b, gv, acc);
                        } else {
                            acc += gv;
                        }
                    }
                }
            }
        }
    }
    part[slice * blockDim.x + threadIdx.x] = acc;
    __syncthreads();
    if (slice == 0 && live) {
        float total_acc = 0.0f;
        for (int j = 0; j < slices; ++j) total_acc += part[j * blockDim.x + threadIdx.x];
        gx[i] = from_f32<T>(total_acc);
    }
}

constexpr int kGw3Stage = 1024;  // (winner, gradient) pairs staged per pass

// grad_w partial sums: block (k*C + c, split) stages the winners and gradients of its share of
// the (n, position) range in shared memory; thread `tap` then walks the staged pairs in order and
// adds the gradients whose winner it is (the pairs are broadcast reads).  part[split][k*C+c][tap]
// receives the min-branch and max-branch sums.
template <typename T>
__global__ void __launch_bounds__(256)
bwd3d_gw_kernel(Geo3 g, int nsplit, const T* __restrict__ gy, const void* __restrict__ winners,
                float* __restrict__ part_min, float* __restrict__ part_max) {
    __shared__ unsigned code_s[kGw3Stage];
    __shared__ float g_s[kGw3Stage];
    const int kc = blockIdx.x, k = kc / g.C, c = kc % g.C, split = blockIdx.y;
    const long long total = (long long)g.N * g.vol;
    const long long per = (total + nsplit - 1) / nsplit;
    const long long j0 = split * per, j1 = min(total, j0 + per);
    const int tap = threadIdx.x;
    float smin = 0.0f, smax = 0.0f;
    for (long long base = j0; base < j1; base += kGw3Stage) {
        const int cnt = (int)min((long long)kGw3Stage, j1 - base);
        __syncthreads();
        for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
            const long long j = base + i;
            const int n = (int)(j / g.vol), pos = (int)(j % g.vol);
            int amn, amx;
            winners3(g, winners, n, k, c, pos, amn, amx);
            code_s[i] = ((unsigned)amn & 0xFFFFu) | ((unsigned)amx << 16);   // -1 stays 0xFFFF: matches no tap
            g_s[i] = to_f32(gy[((size_t)n * g.K + k) * g.vol + pos]);
        }
        __syncthreads();
        if (tap < g.taps) {
            for (int i = 0; i < cnt; ++i) {
                const unsigned code = code_s[i];
                const float gv = g_s[i];
                if ((code & 0xFFFFu) == (unsigned)tap) smin += gv;
                if ((code >> 16) == (unsigned)tap) smax += gv;
            }
        }
    }
    if (tap < g.taps) {
        const size_t o = ((size_t)split * g.K * g.C + kc) * g.taps + tap;
        part_min[o] = smin;
        part_max[o] = smax;
    }
}

// Sums the partials over the splits in order and applies alpha / beta: one thread per (k, c, tap).
__global__ void __launch_bounds__(256)
bwd3d_gw_finish_kernel(Geo3 g, int nsplit, const float* __restrict__ alpha, const float* __restrict__ beta,
                       const float* __restrict__ part_min, const float* __restrict__ part_max,
                       float* __restrict__ gw, float* __restrict__ gw2) {
    const size_t count = (size_t)g.K * g.C * g.taps;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    float tmin = 0.0f, tmax = 0.0f;
    for (int sp = 0; sp < nsplit; ++sp) {
        tmin += part_min[(size_t)sp * count + i];
        tmax += part_max[(size_t)sp * count + i];
    }
    const size_t kc = i / g.taps;
    if (!two_branch(g.mode)) {
        if (gw) gw[i] = (g.mode == TCONV_MIN_PLUS) ? tmin : tmax;
        return;
    }
    const float a = alpha ? alpha[kc] : 1.0f, b = beta ? beta[kc] : 1.0f;
    if (g.mode == TCONV_COMPOUND) {
        if (gw) gw[i] = __fmaf_rn(a, tmin, b * tmax);
    } else {
        if (gw) gw[i] = a * tmin;
        if (gw2) gw2[i] = b * tmax;
    }
}

// grad_alpha / grad_beta partial sums: block (k*C + c, split) sums grad_y * MinPlus3d resp.
// grad_y * MaxPlus3d over its share of the (n, position) range, the branch values rebuilt from the
// winning taps.  part[split][k*C + c][2].
template <typename T>
__global__ void __launch_bounds__(256)
bwd3d_gab_kernel(Geo3 g, int nsplit, const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ w2,
                 const T* __restrict__ gy, const void* __restrict__ winners, float* __restrict__ part) {
    __shared__ float red[256];
    const int c = blockIdx.x % g.C, k = blockIdx.x / g.C, split = blockIdx.y;
    const long long total = (long long)g.N * g.vol;
    const long long per = (total + nsplit - 1) / nsplit;
    const long long j0 = split * per, j1 = min(total, j0 + per);
    const T* wmin = w + ((size_t)k * g.C + c) * g.taps;
    const T* wmax = (g.mode == TCONV_PARALLEL ? w2 : w) + ((size_t)k * g.C + c) * g.taps;
    float sa = 0.0f, sb = 0.0f;
    for (long long j = j0 + threadIdx.x; j < j1; j += blockDim.x) {
        const int n = (int)(j / g.vol), pos = (int)(j % g.vol);
        const int ow = pos % g.OW, oh = (pos / g.OW) % g.OH, od = pos / (g.OW * g.OH);
        int am[2];
        winners3(g, winners, n, k, c, pos, am[0], am[1]);
        const float gv = to_f32(gy[((size_t)n * g.K + k) * g.vol + pos]);
        const T* xc = x + ((size_t)n * g.C + c) * g.D * g.H * g.W;
#pragma unroll
        for (int br = 0; br < 2; ++br) {
            const int tap = am[br];
            const int t = tap / (g.R * g.S), r = (tap / g.S) % g.R, s = tap % g.S;
            const int id = od * g.sd - g.pd + t * g.dd, ih = oh * g.sh - g.ph + r * g.dh,
                      iw = ow * g.sw - g.pw + s * g.dw;
            T xv = zero_of<T>();
            if (id >= 0 && id < g.D && ih >= 0 && ih < g.H && iw >= 0 && iw < g.W)
                xv = xc[((size_t)id * g.H + ih) * g.W + iw];
            const float v = tap_add(xv, br == 0 ? wmin[tap] : wmax[tap]);
            if (br == 0) sa = __fmaf_rn(gv, v, sa); else sb = __fmaf_rn(gv, v, sb);
        }
    }
    const float ta = block_sum(sa, red);
    const float tb = block_sum(sb, red);
    if (threadIdx.x == 0) {
        float* o = part + ((size_t)split * g.K * g.C + blockIdx.x) * 2;
        o[0] = ta;
        o[1] = tb;
    }
}

// grad_bias partial sums: block (k, split); part[split][k].
template <typename T>
__global__ void __launch_bounds__(256)
bwd3d_bias_kernel(Geo3 g, int nsplit, const T* __restrict__ gy, float* __restrict__ part) {
    __shared__ float red[256];
    const int k = blockIdx.x, split = blockIdx.y;
    const long long total = (long long)g.N * g.vol;
    const long long per = (total + nsplit - 1) / nsplit;
    const long long j0 = split * per, j1 = min(total, j0 + per);
    float s = 0.0f;
    for (long long j = j0 + threadIdx.x; j < j1; j += blockDim.x)
        s += to_f32(gy[((size_t)(j / g.vol) * g.K + k) * g.vol + (j % g.vol)]);
    const float t = block_sum(s, red);
    if (threadIdx.x == 0) part[(size_t)split * g.K + k] = t;
}

// Sums partials over the splits in order: out[i] = sum_split part[(split * count + i) * stride + off].
__global__ void __launch_bounds__(256)
bwd3d_sum_splits_kernel(int count, int nsplit, int stride, int off, const float* __restrict__ part,
                        float* __restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    float t = 0.0f;
    for (int sp = 0; sp < nsplit; ++sp) t += part[((size_t)sp * count + i) * stride + off];
    out[i] = t;
}

}  // namespace tconv

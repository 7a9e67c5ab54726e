// Any-shape kernels: one thread per output element (forward), per input element
// (grad_x) or one block per reduced element (parameter gradients).  They accept
// every descriptor the interface allows and serve the shapes the tiled kernels
// do not cover.  All are deterministic and atomic-free.
#pragma once
#include "tconv_common.cuh"

namespace tconv {

// Base operators of Section 3.1 for one (n, k, c, oh, ow): min and max over the
// R x S window of x + w (zero padding), with the lowest winning tap.
template <typename T>
__device__ __forceinline__ void window_generic(const Geo& g, const T* __restrict__ xc,
                                               const T* __restrict__ wmin,
                                               const T* __restrict__ wmax, int oh, int ow,
                                               float& mn, int& amn, float& mx, int& amx) {
    mn = INFINITY;
    mx = -INFINITY;
    amn = 0;
    amx = 0;
    const bool shared_add = (wmin == wmax);
    for (int r = 0; r < g.R; ++r) {
        const int ih = oh * g.sh - g.ph + r * g.dh;
        const bool row_ok = (ih >= 0 && ih < g.H);
        for (int s = 0; s < g.S; ++s) {
            const int iw = ow * g.sw - g.pw + s * g.dw;
            T xv = zero_of<T>();
            if (row_ok && iw >= 0 && iw < g.W) xv = xc[(size_t)ih * g.W + iw];
            else if (g.neutral) continue;    // neutral padding: the tap is skipped
            const int tap = r * g.S + s;
            const float tmn = tap_add(xv, wmin[tap]);
            const float tmx = shared_add ? tmn : tap_add(xv, wmax[tap]);
            if (tmn < mn) { mn = tmn; amn = tap; }
            if (tmx > mx) { mx = tmx; amx = tap; }
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
fwd_generic_kernel(Geo g, const T* __restrict__ x, const T* __restrict__ w,
                   const T* __restrict__ w2, const float* __restrict__ alpha,
                   const float* __restrict__ beta, const float* __restrict__ bias,
                   T* __restrict__ y, void* __restrict__ winners) {
    const size_t total = (size_t)g.N * g.K * g.OH * g.OW;
    const size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= total) return;
    const int ow = (int)(o % g.OW);
    const int oh = (int)((o / g.OW) % g.OH);
    const int k = (int)((o / ((size_t)g.OW * g.OH)) % g.K);
    const int n = (int)(o / ((size_t)g.OW * g.OH * g.K));
    const bool twob = two_branch(g.mode);
    const T* wmin_k = w + (size_t)k * g.C * g.RS;
    const T* wmax_k = (g.mode == TCONV_PARALLEL ? w2 : w) + (size_t)k * g.C * g.RS;
    float best = (g.chan == CH_MAX) ? -INFINITY : INFINITY;
    float acc = 0.0f;
    int win = -1;
    for (int c = 0; c < g.C; ++c) {
        float mn, mx;
        int amn, amx;
        window_generic(g, x + ((size_t)n * g.C + c) * g.H * g.W, wmin_k + (size_t)c * g.RS,
                       wmax_k + (size_t)c * g.RS, oh, ow, mn, amn, mx, amx);
        if (twob) {
            const float a = alpha ? alpha[(size_t)k * g.C + c] : 1.0f;
            const float b = beta ? beta[(size_t)k * g.C + c] : 1.0f;
            acc = __fmaf_rn(a, mn, acc);
            acc = __fmaf_rn(b, mx, acc);
        } else {
            const float m = (g.mode == TCONV_MIN_PLUS) ? mn : mx;
            const int am = (g.mode == TCONV_MIN_PLUS) ? amn : amx;
            if (g.chan == CH_SUM) {
                acc = __fadd_rn(acc, m);
            } else if (g.chan == CH_MAX) {
                if (m > best) { best = m; win = c * g.RS + am; }
            } else {
                if (m < best) { best = m; win = c * g.RS + am; }
            }
            if (g.mode == TCONV_MIN_PLUS) amx = 0; else amn = 0;
        }
        if (winners && g.chan == CH_SUM) {
            const size_t ci = (((size_t)n * g.K + k) * g.C + c) * ((size_t)g.OH * g.OWP) + (size_t)oh * g.OWP + ow;
            if (g.wide) ((uint16_t*)winners)[ci] = (uint16_t)(amn | (amx << 8));
            else ((uint8_t*)winners)[ci] = (uint8_t)(amn | (amx << 4));
            // the row's padding codes (columns OW .. OWP-1) hold tap 0: the backward kernels read whole quads
            if (ow == g.OW - 1)
                for (int pcol = g.OW; pcol < g.OWP; ++pcol) {
                    if (g.wide) ((uint16_t*)winners)[ci + (pcol - ow)] = 0;
                    else ((uint8_t*)winners)[ci + (pcol - ow)] = 0;
                }
        }
    }
    float out = (g.chan == CH_SUM) ? acc : best;
    if (bias) out = __fadd_rn(out, bias[k]);
    if (y) y[o] = from_f32<T>(out);
    if (winners && g.chan != CH_SUM) ((int32_t*)winners)[o] = win;
}

__device__ __forceinline__ void read_code(const Geo& g, const void* winners, size_t ci, int& amn,
                                          int& amx) {
    if (g.wide) {
        const unsigned v = ((const uint16_t*)winners)[ci];
        amn = v & 0xFF;
        amx = v >> 8;
    } else {
        const unsigned v = ((const uint8_t*)winners)[ci];
        amn = v & 0xF;
        amx = v >> 4;
    }
}

// grad_x in gather form: one thread owns one input element and visits, in fixed
// order (k, r, s ascending), every output whose window covers it.
template <typename T>
__global__ void __launch_bounds__(256)
bwd_gx_generic_kernel(Geo g, const float* __restrict__ alpha, const float* __restrict__ beta,
                      const T* __restrict__ gy, const void* __restrict__ winners,
                      T* __restrict__ gx) {
    const size_t total = (size_t)g.N * g.C * g.H * g.W;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int iw = (int)(i % g.W);
    const int ih = (int)((i / g.W) % g.H);
    const int c = (int)((i / ((size_t)g.W * g.H)) % g.C);
    const int n = (int)(i / ((size_t)g.W * g.H * g.C));
    const size_t plane = (size_t)g.OH * g.OW;
    const bool twob = two_branch(g.mode);
    // taps outermost: the output that reads this input through tap (r, s) is found once, then all
    // output channels are visited (fixed order: taps ascending, k ascending inside a tap)
    float acc = 0.0f;
    for (int r = 0; r < g.R; ++r) {
        const int nh = ih + g.ph - r * g.dh;
        if (nh < 0 || nh % g.sh != 0) continue;
        const int oh = nh / g.sh;
        if (oh >= g.OH) continue;
        for (int s = 0; s < g.S; ++s) {
            const int nw = iw + g.pw - s * g.dw;
            if (nw < 0 || nw % g.sw != 0) continue;
            const int ow = nw / g.sw;
            if (ow >= g.OW) continue;
            const int tap = r * g.S + s;
            const size_t op = (size_t)oh * g.OW + ow;
            for (int k = 0; k < g.K; ++k) {
                const size_t obase = ((size_t)n * g.K + k) * plane;
                if (g.chan != CH_SUM) {
                    if (((const int32_t*)winners)[obase + op] == c * g.RS + tap)
                        acc += to_f32(gy[obase + op]);
                } else {
                    const size_t cbase = (((size_t)n * g.K + k) * g.C + c) * ((size_t)g.OH * g.OWP);
                    int amn, amx;
                    read_code(g, winners, cbase + (size_t)oh * g.OWP + ow, amn, amx);
                    const float gv = to_f32(gy[obase + op]);
                    if (twob) {
                        const float a = alpha ? alpha[(size_t)k * g.C + c] : 1.0f;
                        const float b = beta ? beta[(size_t)k * g.C + c] : 1.0f;
                        if (amn == tap) acc = __fmaf_rn(a, gv, acc);
                        if (amx == tap) acc = __fmaf_rn(b, gv, acc);
                    } else if ((g.mode == TCONV_MIN_PLUS ? amn : amx) == tap) {
                        acc += gv;
                    }
                }
            }
        }
    }
    gx[i] = from_f32<T>(acc);
}

// grad_w (and grad_w2): one block per (k, c, tap) sums grad_y over the outputs
// whose winner is that tap.
template <typename T>
__global__ void __launch_bounds__(256)
bwd_gw_generic_kernel(Geo g, const float* __restrict__ alpha, const float* __restrict__ beta,
                      const T* __restrict__ gy, const void* __restrict__ winners,
                      float* __restrict__ gw, float* __restrict__ gw2) {
    __shared__ float red[256];
    const int tap = blockIdx.x % g.RS;
    const int c = (blockIdx.x / g.RS) % g.C;
    const int k = blockIdx.x / (g.RS * g.C);
    const size_t plane = (size_t)g.OH * g.OW;
    const size_t count = (size_t)g.N * plane;
    const bool twob = two_branch(g.mode);
    float smin = 0.0f, smax = 0.0f;
    for (size_t j = threadIdx.x; j < count; j += blockDim.x) {
        const int n = (int)(j / plane);
        const size_t op = j % plane;
        const size_t oi = ((size_t)n * g.K + k) * plane + op;
        if (g.chan != CH_SUM) {
            if (((const int32_t*)winners)[oi] == c * g.RS + tap) smax += to_f32(gy[oi]);
        } else {
            int amn, amx;
            read_code(g, winners, (((size_t)n * g.K + k) * g.C + c) * ((size_t)g.OH * g.OWP) +
                                      (op / g.OW) * g.OWP + op % g.OW, amn, amx);
            const float gv = to_f32(gy[oi]);
            if (twob) {
                if (amn == tap) smin += gv;
                if (amx == tap) smax += gv;
            } else if ((g.mode == TCONV_MIN_PLUS ? amn : amx) == tap) {
                smax += gv;
            }
        }
    }
    const float tmin = block_sum(smin, red);
    const float tmax = block_sum(smax, red);
    if (threadIdx.x == 0) {
        const size_t wi = ((size_t)k * g.C + c) * g.RS + tap;
        if (!twob) {
            if (gw) gw[wi] = tmax;
        } else {
            const float a = alpha ? alpha[(size_t)k * g.C + c] : 1.0f;
            const float b = beta ? beta[(size_t)k * g.C + c] : 1.0f;
            if (g.mode == TCONV_COMPOUND) {
                if (gw) gw[wi] = __fmaf_rn(a, tmin, b * tmax);
            } else {
                if (gw) gw[wi] = a * tmin;
                if (gw2) gw2[wi] = b * tmax;
            }
        }
    }
}

// grad_alpha / grad_beta: one block per (k, c) sums grad_y * MinPlus2d resp.
// grad_y * MaxPlus2d, the branch values rebuilt from the winner codes.
template <typename T>
__global__ void __launch_bounds__(256)
bwd_gab_generic_kernel(Geo g, const T* __restrict__ x, const T* __restrict__ w,
                       const T* __restrict__ w2, const T* __restrict__ gy,
                       const void* __restrict__ winners, float* __restrict__ galpha,
                       float* __restrict__ gbeta) {
    __shared__ float red[256];
    const int c = blockIdx.x % g.C;
    const int k = blockIdx.x / g.C;
    const size_t plane = (size_t)g.OH * g.OW;
    const size_t count = (size_t)g.N * plane;
    const T* wmin = w + ((size_t)k * g.C + c) * g.RS;
    const T* wmax = (g.mode == TCONV_PARALLEL ? w2 : w) + ((size_t)k * g.C + c) * g.RS;
    float sa = 0.0f, sb = 0.0f;
    for (size_t j = threadIdx.x; j < count; j += blockDim.x) {
        const int n = (int)(j / plane);
        const size_t op = j % plane;
        const int oh = (int)(op / g.OW), ow = (int)(op % g.OW);
        int amn, amx;
        read_code(g, winners, (((size_t)n * g.K + k) * g.C + c) * ((size_t)g.OH * g.OWP) + (size_t)oh * g.OWP + ow,
                  amn, amx);
        const float gv = to_f32(gy[((size_t)n * g.K + k) * plane + op]);
        const T* xc = x + ((size_t)n * g.C + c) * g.H * g.W;
        {
            const int ih = oh * g.sh - g.ph + (amn / g.S) * g.dh;
            const int iw = ow * g.sw - g.pw + (amn % g.S) * g.dw;
            T xv = zero_of<T>();
            if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) xv = xc[(size_t)ih * g.W + iw];
            sa = __fmaf_rn(gv, tap_add(xv, wmin[amn]), sa);
        }
        {
            const int ih = oh * g.sh - g.ph + (amx / g.S) * g.dh;
            const int iw = ow * g.sw - g.pw + (amx % g.S) * g.dw;
            T xv = zero_of<T>();
            if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) xv = xc[(size_t)ih * g.W + iw];
            sb = __fmaf_rn(gv, tap_add(xv, wmax[amx]), sb);
        }
    }
    const float ta = block_sum(sa, red);
    const float tb = block_sum(sb, red);
    if (threadIdx.x == 0) {
        if (galpha) galpha[(size_t)k * g.C + c] = ta;
        if (gbeta) gbeta[(size_t)k * g.C + c] = tb;
    }
}

// grad_bias: one block per k.
template <typename T>
__global__ void __launch_bounds__(256)
bwd_bias_kernel(Geo g, const T* __restrict__ gy, float* __restrict__ gbias) {
    __shared__ float red[256];
    const int k = blockIdx.x;
    const size_t plane = (size_t)g.OH * g.OW;
    const size_t count = (size_t)g.N * plane;
    float s = 0.0f;
    for (size_t j = threadIdx.x; j < count; j += blockDim.x) {
        const int n = (int)(j / plane);
        s += to_f32(gy[((size_t)n * g.K + k) * plane + (j % plane)]);
    }
    const float t = block_sum(s, red);
    if (threadIdx.x == 0) gbias[k] = t;
}

// ---------------------------------------------------------------------------------- channel statistics
// sum_y[k], sum_y2[k] = sums over the partial rows (fixed order) of {sum y, sum y^2}: one warp per
// output channel, lane l adds rows l, l + 32, ... in order, then a fixed shuffle tree.
__global__ void __launch_bounds__(256)
stats_finish_kernel(const float* __restrict__ partial, int rows, int pitch, int K, float* __restrict__ sum_y,
                    float* __restrict__ sum_y2) {
    const int k = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (k >= K) return;
    float s1 = 0.0f, s2 = 0.0f;
    for (int r = lane; r < rows; r += 32) {
        const float2 v = *reinterpret_cast<const float2*>(partial + ((size_t)r * pitch + k) * 2);
        s1 += v.x; s2 += v.y;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        s1 += __shfl_xor_sync(0xffffffffu, s1, d);
        s2 += __shfl_xor_sync(0xffffffffu, s2, d);
    }
    if (lane == 0) {
        if (sum_y) sum_y[k] = s1;
        if (sum_y2) sum_y2[k] = s2;
    }
}

// Statistics of a stored output (layers the tiled kernels do not serve): grid (K, chunks of images),
// partial[chunk][k] = {sum y, sum y^2} over the chunk.
template <typename T>
__global__ void __launch_bounds__(256)
stats_direct_kernel(Geo g, const T* __restrict__ y, float* __restrict__ partial, int n_per_chunk) {
    __shared__ float red[256];
    const int k = blockIdx.x, chunk = blockIdx.y;
    const size_t plane = (size_t)g.OH * g.OW;
    const int n_lo = chunk * n_per_chunk, n_hi = min(g.N, n_lo + n_per_chunk);
    float s1 = 0.0f, s2 = 0.0f;
    for (int n = n_lo; n < n_hi; ++n) {
        const T* src = y + ((size_t)n * g.K + k) * plane;
        for (size_t j = threadIdx.x; j < plane; j += blockDim.x) {
            const float v = to_f32(src[j]);
            s1 += v; s2 = __fmaf_rn(v, v, s2);
        }
    }
    const float t1 = block_sum(s1, red);
    const float t2 = block_sum(s2, red);
    if (threadIdx.x == 0) *reinterpret_cast<float2*>(partial + ((size_t)chunk * g.K + k) * 2) = make_float2(t1, t2);
}

}  // namespace tconv

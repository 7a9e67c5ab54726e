// Depthwise (groups = C) tropical convolution: every channel is its own group,
//   y[n][c] = alpha[c] * min_tap(x[n][c] + w[c]) + beta[c] * max_tap(x[n][c] + w2[c]) + bias[c]
// (max_plus / min_plus: the one extremum; compound: w2 = w).  Nine taps per output put this
// form on the memory roofline: x is read once (through L1 / L2 for the window overlap), y and,
// on request, one winner byte per output are written once.
// Weights are [C][R][S]; alpha, beta, bias [C]; winner codes uint8 [N][C][OH][OW] with the argmin
// tap in the low nibble and the argmax tap in the high nibble (R * S <= 16).
#pragma once
#include "tconv_common.cuh"

namespace tconv {

// ---------------------------------------------------------------------------------- forward
// One thread per quad of 4 horizontally adjacent outputs of one (n, c) plane; consecutive
// threads own consecutive quads, so a warp reads contiguous pieces of up to R input rows.
template <typename T, int MODE, bool WIN>
__global__ void __launch_bounds__(256)
dw_fwd_kernel(Geo g, const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ w2,
              const float* __restrict__ alpha, const float* __restrict__ beta,
              const float* __restrict__ bias, T* __restrict__ y, uint8_t* __restrict__ codes,
              int QPR, size_t total_quads) {
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool PAR = (MODE == TCONV_PARALLEL);
    constexpr bool DO_MIN = TWO || MODE == TCONV_MIN_PLUS, DO_MAX = TWO || MODE == TCONV_MAX_PLUS;
    // (the host rejects layers whose quad or element counts do not fit 31 bits)
    const unsigned q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= total_quads) return;
    const unsigned t = q / (unsigned)QPR;
    const int qx = (int)(q - t * (unsigned)QPR);
    const size_t nc = t / (unsigned)g.OH;
    const int oh = (int)(t - (unsigned)nc * (unsigned)g.OH);
    const int c = (int)((unsigned)nc % (unsigned)g.C);
    const int ow0 = qx * 4;
    const T* xp = x + nc * (size_t)g.H * g.W;
    const T* wc = w + (size_t)c * g.RS;
    const T* wc2 = PAR ? w2 + (size_t)c * g.RS : wc;
    float mn[4], mx[4];
    int amn[4], amx[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) { mn[j] = INFINITY; mx[j] = -INFINITY; amn[j] = 0; amx[j] = 0; }
    const int ih0 = oh * g.sh - g.ph;
    const int iw0 = ow0 * g.sw - g.pw;
    for (int r = 0; r < g.R; ++r) {
        const int ih = ih0 + r * g.dh;
        const bool row_ok = ih >= 0 && ih < g.H;
        const T* xr = xp + (size_t)(row_ok ? ih : 0) * g.W;
        for (int s = 0; s < g.S; ++s) {
            const int tap = r * g.S + s;
            const T wv = __ldg(wc + tap);
            const T wv2 = PAR ? __ldg(wc2 + tap) : wv;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int iw = iw0 + j * g.sw + s * g.dw;
                const T xv = (row_ok && iw >= 0 && iw < g.W) ? __ldg(xr + iw) : zero_of<T>();
                const float ta = tap_add(xv, wv);
                const float tb = PAR ? tap_add(xv, wv2) : ta;
                if constexpr (WIN) {
                    // strict compares in ascending tap order: the lowest tap wins a tie
                    if (DO_MIN && ta < mn[j]) { mn[j] = ta; amn[j] = tap; }
                    if (DO_MAX && tb > mx[j]) { mx[j] = tb; amx[j] = tap; }
                } else {
                    if (DO_MIN) mn[j] = fminf(mn[j], ta);
                    if (DO_MAX) mx[j] = fmaxf(mx[j], tb);
                }
            }
        }
    }
    const float a = (TWO && alpha) ? alpha[c] : 1.0f, b = (TWO && beta) ? beta[c] : 1.0f;
    const float bk = bias ? bias[c] : 0.0f;
    const size_t o = (nc * g.OH + oh) * (size_t)g.OW + ow0;
    const bool full = (ow0 + 3 < g.OW) && ((g.OW & 3) == 0);
    if (y) {
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // same evaluation order as the dense Sum forms with one channel: the sum starts at 0
            float acc;
            if constexpr (TWO) acc = __fmaf_rn(b, mx[j], __fmaf_rn(a, mn[j], 0.0f));
            else acc = __fadd_rn(0.0f, DO_MIN ? mn[j] : mx[j]);
            v[j] = bias ? __fadd_rn(acc, bk) : acc;
        }
        if (full) {
            if constexpr (sizeof(T) == 4) {
                *reinterpret_cast<float4*>(y + o) = make_float4(v[0], v[1], v[2], v[3]);
            } else {
                const __nv_bfloat162 p01 = __floats2bfloat162_rn(v[0], v[1]);
                const __nv_bfloat162 p23 = __floats2bfloat162_rn(v[2], v[3]);
                *reinterpret_cast<uint2*>(y + o) = make_uint2(*reinterpret_cast<const unsigned*>(&p01),
                                                              *reinterpret_cast<const unsigned*>(&p23));
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (ow0 + j < g.OW) y[o + j] = from_f32<T>(v[j]);
        }
    }
    if constexpr (WIN) {
        unsigned packed = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const unsigned code = (DO_MIN ? (unsigned)amn[j] : 0u) | (DO_MAX ? (unsigned)amx[j] << 4 : 0u);
            packed |= code << (8 * j);
        }
        if (full) {
            *reinterpret_cast<unsigned*>(codes + o) = packed;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (ow0 + j < g.OW) codes[o + j] = (uint8_t)(packed >> (8 * j));
        }
    }
}

// ---------------------------------------------------------------------------------- grad_x
// Gather form: one thread per input element visits, in ascending tap order, the outputs that read
// it, and takes coef * grad_y from those whose winner is that tap.  No atomics, fixed order.
// BR: 0 both branches, 1 min branch only, 2 max branch only.
template <typename T, int BR>
__global__ void __launch_bounds__(256)
dw_bwd_gx_kernel(Geo g, const float* __restrict__ alpha, const float* __restrict__ beta,
                 const T* __restrict__ gy, const uint8_t* __restrict__ codes, T* __restrict__ gx,
                 size_t total) {
    const unsigned i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const unsigned t = i / (unsigned)g.W;
    const int iw = (int)(i - t * (unsigned)g.W);
    const size_t nc = t / (unsigned)g.H;
    const int ih = (int)(t - (unsigned)nc * (unsigned)g.H);
    const int c = (int)((unsigned)nc % (unsigned)g.C);
    const float a = (BR == 0 && alpha) ? alpha[c] : 1.0f, b = (BR == 0 && beta) ? beta[c] : 1.0f;
    const T* gp = gy + nc * (size_t)g.OH * g.OW;
    const uint8_t* cp = codes + nc * (size_t)g.OH * g.OW;
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
            const unsigned tap = (unsigned)(r * g.S + s);
            const unsigned code = __ldg(cp + (size_t)oh * g.OW + ow);
            const float gv = to_f32(__ldg(gp + (size_t)oh * g.OW + ow));
            if ((BR == 0 || BR == 1) && (code & 15u) == tap) acc = (BR == 0) ? __fmaf_rn(a, gv, acc) : acc + gv;
            if ((BR == 0 || BR == 2) && (code >> 4) == tap) acc = (BR == 0) ? __fmaf_rn(b, gv, acc) : acc + gv;
        }
    }
    gx[i] = from_f32<T>(acc);
}

// ---------------------------------------------------------------------------------- parameter gradients
// Per channel: G_min[tap], G_max[tap] = sum of grad_y over the outputs whose min / max winner is
// tap; A = sum grad_y * min value, B = sum grad_y * max value (the branch values are rebuilt as
// x[winner] + w[winner]); S = sum grad_y.  CTA (c, chunk) walks its share of the channel's
// (n, oh, ow) items with per-thread private columns in shared memory, reduces them in a fixed
// order and writes one partial row; dw_bwd_finish_kernel sums the chunks in order.
constexpr int kDwAcc = 2 * 16 + 3;   // accumulators per channel: G_min[16], G_max[16], A, B, S

template <typename T, int BR, bool PAR>
__global__ void __launch_bounds__(256)
dw_bwd_params_kernel(Geo g, const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ w2,
                     const T* __restrict__ gy, const uint8_t* __restrict__ codes,
                     float* __restrict__ partial, int nchunks, int need_ab) {
    extern __shared__ float col[];   // [kDwAcc][256]
    const int c = blockIdx.x, chunk = blockIdx.y, tid = threadIdx.x;
    for (int e = tid; e < kDwAcc * 256; e += 256) col[e] = 0.0f;
    __syncthreads();
    const unsigned plane = (unsigned)g.OH * g.OW;
    const unsigned items = (unsigned)g.N * plane;
    const unsigned per = (items + nchunks - 1) / nchunks;
    const unsigned lo = min(items, (unsigned)chunk * per), hi = min(items, lo + per);
    const T* wc = w + (size_t)c * g.RS;
    const T* wc2 = PAR ? w2 + (size_t)c * g.RS : wc;
    float* mine = col + tid;
    for (unsigned it = lo + tid; it < hi; it += 256) {
        const unsigned n = it / plane;
        const unsigned pix = it - n * plane;
        const int oh = (int)(pix / (unsigned)g.OW), ow = (int)(pix - (unsigned)oh * (unsigned)g.OW);
        const size_t o = ((size_t)n * g.C + c) * plane + pix;
        const float gv = to_f32(__ldg(gy + o));
        const unsigned code = __ldg(codes + o);
        const T* xp = x + ((size_t)n * g.C + c) * (size_t)g.H * g.W;
        mine[(2 * 16 + 2) * 256] += gv;
        if (BR == 0 || BR == 1) {
            const unsigned tp = code & 15u;
            mine[tp * 256] += gv;
            if (need_ab) {
                const int ih = oh * g.sh - g.ph + (int)(tp / g.S) * g.dh, iw = ow * g.sw - g.pw + (int)(tp % g.S) * g.dw;
                const T xv = (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) ? __ldg(xp + (size_t)ih * g.W + iw) : zero_of<T>();
                mine[(2 * 16) * 256] = __fmaf_rn(gv, tap_add(xv, __ldg(wc + tp)), mine[(2 * 16) * 256]);
            }
        }
        if (BR == 0 || BR == 2) {
            const unsigned tp = code >> 4;
            mine[(16 + tp) * 256] += gv;
            if (need_ab) {
                const int ih = oh * g.sh - g.ph + (int)(tp / g.S) * g.dh, iw = ow * g.sw - g.pw + (int)(tp % g.S) * g.dw;
                const T xv = (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) ? __ldg(xp + (size_t)ih * g.W + iw) : zero_of<T>();
                mine[(2 * 16 + 1) * 256] = __fmaf_rn(gv, tap_add(xv, __ldg(wc2 + tp)), mine[(2 * 16 + 1) * 256]);
            }
        }
    }
    __syncthreads();
    // row a of the columns is summed by warp a % 8: 8 values per lane in order, then a fixed shuffle tree
    const int warp = tid >> 5, lane = tid & 31;
    for (int a = warp; a < kDwAcc; a += 8) {
        float s = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) s += col[a * 256 + lane * 8 + e];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) s += __shfl_down_sync(0xffffffffu, s, d);
        if (lane == 0) partial[((size_t)chunk * g.C + c) * kDwAcc + a] = s;
    }
}

// One thread per (c, accumulator): sums the chunk partials in order and writes the gradients.
__global__ void dw_bwd_finish_kernel(Geo g, const float* __restrict__ partial, int nchunks, int mode,
                                     const float* __restrict__ alpha, const float* __restrict__ beta,
                                     float* __restrict__ gw, float* __restrict__ gw2,
                                     float* __restrict__ galpha, float* __restrict__ gbeta,
                                     float* __restrict__ gbias) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= g.C * kDwAcc) return;
    const int c = i / kDwAcc, a = i - c * kDwAcc;
    float s = 0.0f;
    for (int ch = 0; ch < nchunks; ++ch) s += partial[((size_t)ch * g.C + c) * kDwAcc + a];
    const bool two = two_branch(mode);
    const float al = (two && alpha) ? alpha[c] : 1.0f, be = (two && beta) ? beta[c] : 1.0f;
    if (a == 2 * 16 + 2) { if (gbias) gbias[c] = s; return; }
    if (a == 2 * 16) { if (two && galpha) galpha[c] = s; return; }
    if (a == 2 * 16 + 1) { if (two && gbeta) gbeta[c] = s; return; }
    const int tap = a & 15;
    if (tap >= g.RS) return;
    // grad_w takes the min branch (and, outside parallel mode, the max branch too, summed below by
    // the thread of the min-branch accumulator); grad_w2 takes the max branch of parallel mode
    if (a < 16) {
        if (!gw) return;
        float v = (mode == TCONV_MAX_PLUS) ? 0.0f : al * s;
        if (mode == TCONV_MAX_PLUS || mode == TCONV_COMPOUND) {
            float smax = 0.0f;
            for (int ch = 0; ch < nchunks; ++ch) smax += partial[((size_t)ch * g.C + c) * kDwAcc + 16 + tap];
            v = (mode == TCONV_MAX_PLUS) ? smax : __fmaf_rn(be, smax, v);
        }
        gw[(size_t)c * g.RS + tap] = v;
    } else if (mode == TCONV_PARALLEL && gw2) {
        gw2[(size_t)c * g.RS + tap] = be * s;
    }
}

}  // namespace tconv

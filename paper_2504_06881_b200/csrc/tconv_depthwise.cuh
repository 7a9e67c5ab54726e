// Depthwise (groups = C) tropical convolution: every channel is its own group,
//   y[n][c] = alpha[c] * min_tap(x[n][c] + w[c]) + beta[c] * max_tap(x[n][c] + w2[c]) + bias[c]
// (max_plus / min_plus: the one extremum; compound: w2 = w).  Nine taps per output put this
// form on the memory roofline: x is read once (through L1 / L2 for the window overlap), y and,
// on request, one winner byte per output are written once.
// Weights are [C][R][S]; alpha, beta, bias [C]; winner codes uint8 [N][C][OH][OW] with the argmin
// tap in the low nibble and the argmax tap in the high nibble (R * S <= 16).
#pragma once
#include "tconv_common.cuh"
#include "tconv_tiled.cuh"   // ext3 (3-input min / max)

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

// ---------------------------------------------------------------------------------- forward, 3x3 windows
// extremum of nine values with 3-input min / max (3 + 2 + 2 + 2)
__device__ __forceinline__ float dw_fold9(const float* v, bool is_min) {
    float m = ext3(v[0], v[1], v[2], is_min);
    m = ext3(m, v[3], v[4], is_min);
    m = ext3(m, v[5], v[6], is_min);
    return ext3(m, v[7], v[8], is_min);
}
__device__ __forceinline__ void load4(const float* p, float* out) {
    const float4 v = __ldg(reinterpret_cast<const float4*>(p));
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, __nv_bfloat16* out) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&v.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&v.y);
    out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
}
// L consecutive elements of a row, starting at column c0, in a single code path: bit i of `mask`
// says whether column c0 + i lies inside the row (computed once per thread); `rp` points at column
// c0 of the row (it is dereferenced only where the mask allows); a row outside the plane
// (row_ok false) reads as zero.  VEC: c0 + 1 is a multiple of 4 and rows start on 4-element
// boundaries, so every group of 4 from c0 + 1 on is wholly inside or wholly outside the row and
// is read with one aligned load.
__device__ __forceinline__ unsigned dw_col_mask(int c0, int L, int W) {
    unsigned m = 0;
    for (int i = 0; i < L; ++i)
        if (c0 + i >= 0 && c0 + i < W) m |= 1u << i;
    return m;
}
template <typename T, int L, bool VEC>
__device__ __forceinline__ void dw_load_row(const T* rp, bool row_ok, unsigned mask, T* out) {
    if (!row_ok) mask = 0;
    if constexpr (VEC) {
        out[0] = (mask & 1u) ? __ldg(rp) : zero_of<T>();
#pragma unroll
        for (int i = 1; i + 4 <= L; i += 4) {
            if ((mask >> i) & 1u) {
                load4(rp + i, out + i);
            } else {
                out[i] = out[i + 1] = out[i + 2] = out[i + 3] = zero_of<T>();
            }
        }
#pragma unroll
        for (int i = 1 + ((L - 1) / 4) * 4; i < L; ++i) out[i] = ((mask >> i) & 1u) ? __ldg(rp + i) : zero_of<T>();
    } else {
#pragma unroll
        for (int i = 0; i < L; ++i) out[i] = ((mask >> i) & 1u) ? __ldg(rp + i) : zero_of<T>();
    }
}

// 3x3 window, dilation 1, stride SW in both directions.  A thread owns a strip of 4 output
// columns x RT output rows of one (n, c) plane and slides a window of three input rows held in
// registers down the strip: every input row of the strip is loaded once per thread.  The nine
// weights of the channel sit in registers.
constexpr int kDwRT = 6;   // output rows per strip of the 3x3 depthwise kernels
constexpr int kDwAhead = 3;   // output rows by which the forward strip kernels request their input rows ahead

template <typename T, int MODE, bool WIN, int SW, bool VEC>
__global__ void __launch_bounds__(256)
dw_fwd3_kernel(Geo g, const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ w2,
               const float* __restrict__ alpha, const float* __restrict__ beta,
               const float* __restrict__ bias, T* __restrict__ y, uint8_t* __restrict__ codes,
               int QPR, int strips, unsigned total) {
    constexpr int RT = kDwRT;             // output rows per strip
    constexpr int L = 3 * SW + 3;               // input columns 4 outputs touch
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool PAR = (MODE == TCONV_PARALLEL);
    constexpr bool DO_MIN = TWO || MODE == TCONV_MIN_PLUS, DO_MAX = TWO || MODE == TCONV_MAX_PLUS;
    const unsigned q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= total) return;
    const unsigned t = q / (unsigned)QPR;
    const int qx = (int)(q - t * (unsigned)QPR);
    const size_t nc = t / (unsigned)strips;
    const int oh0 = (int)(t - (unsigned)nc * (unsigned)strips) * RT;
    const int c = (int)((unsigned)nc % (unsigned)g.C);
    const int ow0 = qx * 4;
    const T* xp = x + nc * (size_t)g.H * g.W;
    T wa[9], wb[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) {
        wa[i] = __ldg(w + (size_t)c * 9 + i);
        wb[i] = PAR ? __ldg(w2 + (size_t)c * 9 + i) : wa[i];
    }
    const float a = (TWO && alpha) ? alpha[c] : 1.0f, b = (TWO && beta) ? beta[c] : 1.0f;
    const float bk = bias ? bias[c] : 0.0f;
    const int ih0 = oh0 * SW - g.ph, c0 = ow0 * SW - g.pw;
    const bool full = (ow0 + 3 < g.OW) && ((g.OW & 3) == 0);
    // input row rho of the strip lives in win[rho % WR]; the rows that output row k + AH needs
    // first are requested before output row k is computed
    constexpr int AH = SW == 1 ? kDwAhead : 1;   // stride 2: a row is nine registers, one row ahead
    constexpr int WR = 3 + AH * SW;
    T win[WR][L];
    const unsigned cmask = dw_col_mask(c0, L, g.W);
    const T* rp0 = xp + (ptrdiff_t)ih0 * g.W + c0;   // column c0 of the strip's first input row
    auto load = [&](int rho) {
        const int ih = ih0 + rho;
        dw_load_row<T, L, VEC>(rp0 + rho * g.W, ih >= 0 && ih < g.H, cmask, win[rho % WR]);
    };
#pragma unroll
    for (int rho = 0; rho <= (AH - 1) * SW + 2; ++rho) load(rho);
#pragma unroll
    for (int k = 0; k < RT; ++k) {
        if (oh0 + k >= g.OH) break;
        if (k + AH < RT) {
#pragma unroll
            for (int rho = (k + AH - 1) * SW + 3; rho <= (k + AH) * SW + 2; ++rho) load(rho);
        }
        // per pixel: nine tap sums, their extrema with 3-input min / max and, for the winner codes,
        // the first tap that attains each extremum, recovered on the FMA pipe: d = (t - m) * 2^32 is
        // zero exactly for winning taps, key = |d| * (-2^125) + (2^23 + rank) is 2^23 + rank for them
        // and below 2^23 otherwise, the largest key belongs to the lowest winning tap and carries
        // rank = 15 - tap (min branch) or 16 * (15 - tap) (max branch) in its low mantissa bits
        // (|x + w| < 2^95 assumed)
        float mn[4], mx[4];
        unsigned code4[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float ta[9], tb[PAR ? 9 : 1];
#pragma unroll
            for (int tap = 0; tap < 9; ++tap) {
                const T xv = win[(k * SW + tap / 3) % WR][j * SW + tap % 3];
                ta[tap] = tap_add(xv, wa[tap]);
                if constexpr (PAR) tb[tap] = tap_add(xv, wb[tap]);
            }
            const float* tm = PAR ? tb : ta;
            if constexpr (DO_MIN) mn[j] = dw_fold9(ta, true);
            if constexpr (DO_MAX) mx[j] = dw_fold9(tm, false);
            if constexpr (WIN) {
                constexpr float kS = 4294967296.0f, kH = 4.253529586511731e37f, kB = 8388608.0f;
                unsigned bmn = 0u, bmx = 0u;
                if constexpr (DO_MIN) {
                    const float e = -mn[j] * kS;
                    float key[9];
#pragma unroll
                    for (int tap = 0; tap < 9; ++tap)
                        key[tap] = __fmaf_rn(-kH, __fmaf_rn(kS, ta[tap], e), kB + (float)(15 - tap));
                    bmn = __float_as_uint(dw_fold9(key, false));
                }
                if constexpr (DO_MAX) {
                    const float e = -mx[j] * kS;
                    float key[9];
#pragma unroll
                    for (int tap = 0; tap < 9; ++tap)
                        key[tap] = __fmaf_rn(kH, __fmaf_rn(kS, tm[tap], e), kB + (float)(16 * (15 - tap)));
                    bmx = __float_as_uint(dw_fold9(key, false));
                }
                code4[j] = (DO_MIN ? (~bmn & 0x0fu) : 0u) | (DO_MAX ? (~bmx & 0xf0u) : 0u);
            }
        }
        const size_t o = (nc * g.OH + oh0 + k) * (size_t)g.OW + ow0;
        if (y) {
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
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
            const unsigned packed = code4[0] | (code4[1] << 8) | (code4[2] << 16) | (code4[3] << 24);
            if (full) {
                *reinterpret_cast<unsigned*>(codes + o) = packed;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (ow0 + j < g.OW) codes[o + j] = (uint8_t)(packed >> (8 * j));
            }
        }
    }
}

// ---------------------------------------------------------------------------------- forward, 3x3, bf16 pairs
// bf16, stride 1: the strip kernel above on packed pairs.  A 32-bit register holds the inputs of
// two horizontally adjacent outputs; an input row of the strip is kept as the five pairs (e0,e1),
// (e1,e2), ..., (e4,e5) of its six columns, so that tap column s of output pair p is pair 2p + s.
// One add.bf16x2 forms two tap sums (each one rounded bf16 add), min / max.bf16x2 fold them (exact),
// the two-branch combine runs in fp32.  Winner codes: taps descending, a per-half equality mask
// against the extremum selects the tap, so the lowest equal tap stays.
__device__ __forceinline__ unsigned dw_hadd2(unsigned a, unsigned b) {
    unsigned d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ unsigned dw_hmin2(unsigned a, unsigned b) {
    unsigned d;
    asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ unsigned dw_hmax2(unsigned a, unsigned b) {
    unsigned d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ unsigned dw_fold9_h2(const unsigned* v, bool is_min) {
    unsigned m = v[0];
#pragma unroll
    for (int i = 1; i < 9; ++i) m = is_min ? dw_hmin2(m, v[i]) : dw_hmax2(m, v[i]);
    return m;
}
__device__ __forceinline__ unsigned dw_heq2_mask(unsigned a, unsigned b) {
    return __heq2_mask(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
}

template <int MODE, bool WIN, bool VEC>
__global__ void __launch_bounds__(256)
dw_fwd3_bf16_kernel(Geo g, const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                    const __nv_bfloat16* __restrict__ w2, const float* __restrict__ alpha,
                    const float* __restrict__ beta, const float* __restrict__ bias,
                    __nv_bfloat16* __restrict__ y, uint8_t* __restrict__ codes, int QPR, int strips,
                    unsigned total) {
    using T = __nv_bfloat16;
    constexpr int RT = kDwRT, L = 6;
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool PAR = (MODE == TCONV_PARALLEL);
    constexpr bool DO_MIN = TWO || MODE == TCONV_MIN_PLUS, DO_MAX = TWO || MODE == TCONV_MAX_PLUS;
    const unsigned q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= total) return;
    const unsigned t = q / (unsigned)QPR;
    const int qx = (int)(q - t * (unsigned)QPR);
    const size_t nc = t / (unsigned)strips;
    const int oh0 = (int)(t - (unsigned)nc * (unsigned)strips) * RT;
    const int c = (int)((unsigned)nc % (unsigned)g.C);
    const int ow0 = qx * 4;
    const T* xp = x + nc * (size_t)g.H * g.W;
    unsigned wa[9], wb[9];   // {w, w}
#pragma unroll
    for (int i = 0; i < 9; ++i) {
        wa[i] = 0x00010001u * (unsigned)__bfloat16_as_ushort(__ldg(w + (size_t)c * 9 + i));
        wb[i] = PAR ? 0x00010001u * (unsigned)__bfloat16_as_ushort(__ldg(w2 + (size_t)c * 9 + i)) : wa[i];
    }
    const float a = (TWO && alpha) ? alpha[c] : 1.0f, b = (TWO && beta) ? beta[c] : 1.0f;
    const float bk = bias ? bias[c] : 0.0f;
    const int ih0 = oh0 - g.ph, c0 = ow0 - g.pw;
    const bool full = (ow0 + 3 < g.OW) && ((g.OW & 3) == 0);
    // Rows are requested kDwAhead output rows ahead into a ring of raw loads (first column, the four
    // aligned columns as two words, last column) and turned into the five pairs when they enter the
    // window of three rows, win[rho % 3].
    constexpr int RW = kDwAhead + 1;
    static_assert(kDwAhead >= 2, "row k + 2 must have been requested before output row k");
    unsigned raw[RW][4];
    unsigned win[3][5];
    const unsigned cmask = dw_col_mask(c0, L, g.W);
    const T* rp0 = xp + (ptrdiff_t)ih0 * g.W + c0;
    auto issue = [&](int rho) {
        const int ih = ih0 + rho;
        const unsigned mask = (ih >= 0 && ih < g.H) ? cmask : 0u;
        const unsigned short* rp = reinterpret_cast<const unsigned short*>(rp0 + rho * g.W);
        unsigned* r = raw[rho % RW];
        if constexpr (VEC) {
            r[0] = (mask & 1u) ? (unsigned)__ldg(rp) : 0u;
            if ((mask >> 1) & 1u) {
                const uint2 v = __ldg(reinterpret_cast<const uint2*>(rp + 1));
                r[1] = v.x;
                r[2] = v.y;
            } else {
                r[1] = r[2] = 0u;
            }
            r[3] = ((mask >> 5) & 1u) ? (unsigned)__ldg(rp + 5) : 0u;
        } else {
            unsigned e[L];
#pragma unroll
            for (int i = 0; i < L; ++i) e[i] = ((mask >> i) & 1u) ? (unsigned)__ldg(rp + i) : 0u;
            r[0] = e[0];
            r[1] = e[1] | (e[2] << 16);
            r[2] = e[3] | (e[4] << 16);
            r[3] = e[5];
        }
    };
    auto pack = [&](int rho) {
        const unsigned* r = raw[rho % RW];
        unsigned* d = win[rho % 3];
        d[0] = __byte_perm(r[0], r[1], 0x5410);
        d[1] = r[1];
        d[2] = __byte_perm(r[1], r[2], 0x5432);
        d[3] = r[2];
        d[4] = __byte_perm(r[2], r[3], 0x5432);
    };
#pragma unroll
    for (int rho = 0; rho <= kDwAhead; ++rho) issue(rho);
    pack(0);
    pack(1);
#pragma unroll
    for (int k = 0; k < RT; ++k) {
        if (oh0 + k >= g.OH) break;
        pack(k + 2);
        if (k + kDwAhead <= RT) issue(k + kDwAhead + 1);
        float mn[4], mx[4];
        unsigned code2[2] = {0u, 0u};
#pragma unroll
        for (int pr = 0; pr < 2; ++pr) {
            unsigned ta[9], tb[PAR ? 9 : 1];
#pragma unroll
            for (int tap = 0; tap < 9; ++tap) {
                const unsigned xv = win[(k + tap / 3) % 3][2 * pr + tap % 3];
                ta[tap] = dw_hadd2(xv, wa[tap]);
                if constexpr (PAR) tb[tap] = dw_hadd2(xv, wb[tap]);
            }
            const unsigned* tm = PAR ? tb : ta;
            unsigned m2 = 0u, M2 = 0u;
            if constexpr (DO_MIN) {
                m2 = dw_fold9_h2(ta, true);
                mn[2 * pr] = __uint_as_float(m2 << 16);
                mn[2 * pr + 1] = __uint_as_float(m2 & 0xffff0000u);
            }
            if constexpr (DO_MAX) {
                M2 = dw_fold9_h2(tm, false);
                mx[2 * pr] = __uint_as_float(M2 << 16);
                mx[2 * pr + 1] = __uint_as_float(M2 & 0xffff0000u);
            }
            if constexpr (WIN) {
                unsigned smn = 0u, smx = 0u;
#pragma unroll
                for (int tap = 8; tap >= 0; --tap) {
                    if constexpr (DO_MIN) {
                        const unsigned eq = dw_heq2_mask(ta[tap], m2);
                        smn = (eq & (0x00010001u * (unsigned)tap)) | (~eq & smn);
                    }
                    if constexpr (DO_MAX) {
                        const unsigned eq = dw_heq2_mask(tm[tap], M2);
                        smx = (eq & (0x00010001u * (unsigned)tap)) | (~eq & smx);
                    }
                }
                code2[pr] = smn | (smx << 4);
            }
        }
        const size_t o = (nc * g.OH + oh0 + k) * (size_t)g.OW + ow0;
        if (y) {
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float acc;
                if constexpr (TWO) acc = __fmaf_rn(b, mx[j], __fmaf_rn(a, mn[j], 0.0f));
                else acc = __fadd_rn(0.0f, DO_MIN ? mn[j] : mx[j]);
                v[j] = bias ? __fadd_rn(acc, bk) : acc;
            }
            if (full) {
                const __nv_bfloat162 p01 = __floats2bfloat162_rn(v[0], v[1]);
                const __nv_bfloat162 p23 = __floats2bfloat162_rn(v[2], v[3]);
                *reinterpret_cast<uint2*>(y + o) = make_uint2(*reinterpret_cast<const unsigned*>(&p01),
                                                              *reinterpret_cast<const unsigned*>(&p23));
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (ow0 + j < g.OW) y[o + j] = __float2bfloat16_rn(v[j]);
            }
        }
        if constexpr (WIN) {
            // bytes 0 and 2 of each pair's code word are the codes of its two outputs
            const unsigned packed = __byte_perm(code2[0], code2[1], 0x6420);
            if (full) {
                *reinterpret_cast<unsigned*>(codes + o) = packed;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (ow0 + j < g.OW) codes[o + j] = (uint8_t)(packed >> (8 * j));
            }
        }
    }
}

// ---------------------------------------------------------------------------------- grad_x, 3x3 at stride 2
// 3x3 window, stride 2, padding 1, dilation 1: the outputs that read an input element, and through
// which tap, depend only on the parity of its row and column.  One thread owns the 2 x 2 input block
// (2a, 2b) .. (2a + 1, 2b + 1) and the four outputs (a, b) .. (a + 1, b + 1) that reach it:
//   (2a,   2b  ): (a, b) tap 4
//   (2a,   2b+1): (a, b+1) tap 3, (a, b) tap 5
//   (2a+1, 2b  ): (a+1, b) tap 1, (a, b) tap 7
//   (2a+1, 2b+1): (a+1, b+1) tap 0, (a+1, b) tap 2, (a, b+1) tap 6, (a, b) tap 8
// Every thread runs the same nine comparisons per branch, in ascending tap order per element.
// BR: 0 both branches, 1 min branch only, 2 max branch only.
template <typename T, int BR>
__global__ void __launch_bounds__(256)
dw_bwd_gx_s2_kernel(Geo g, const float* __restrict__ alpha, const float* __restrict__ beta,
                    const T* __restrict__ gy, const uint8_t* __restrict__ codes, T* __restrict__ gx,
                    int HB, int WB, unsigned total) {
    const unsigned i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const unsigned t = i / (unsigned)WB;
    const int b = (int)(i - t * (unsigned)WB);
    const size_t nc = t / (unsigned)HB;
    const int a = (int)(t - (unsigned)nc * (unsigned)HB);
    const int c = (int)((unsigned)nc % (unsigned)g.C);
    const float ca = (BR == 0 && alpha) ? alpha[c] : 1.0f, cb = (BR == 0 && beta) ? beta[c] : 1.0f;
    const T* gp = gy + nc * (size_t)g.OH * g.OW;
    const uint8_t* cp = codes + nc * (size_t)g.OH * g.OW;
    // the four outputs; one outside the map gets a code no tap equals
    unsigned code[2][2];
    float gv[2][2];
#pragma unroll
    for (int da = 0; da < 2; ++da)
#pragma unroll
        for (int db = 0; db < 2; ++db) {
            const int oh = a + da, ow = b + db;
            const bool ok = oh < g.OH && ow < g.OW;
            code[da][db] = ok ? (unsigned)__ldg(cp + (size_t)oh * g.OW + ow) : 0xffu;
            gv[da][db] = ok ? to_f32(__ldg(gp + (size_t)oh * g.OW + ow)) : 0.0f;
        }
    auto take = [&](float acc, int da, int db, unsigned tap) {
        const unsigned cd = code[da][db];
        const float v = gv[da][db];
        if ((BR == 0 || BR == 1) && (cd & 15u) == tap) acc = (BR == 0) ? __fmaf_rn(ca, v, acc) : acc + v;
        if ((BR == 0 || BR == 2) && (cd >> 4) == tap) acc = (BR == 0) ? __fmaf_rn(cb, v, acc) : acc + v;
        return acc;
    };
    const float e00 = take(0.0f, 0, 0, 4u);
    const float e01 = take(take(0.0f, 0, 1, 3u), 0, 0, 5u);
    const float e10 = take(take(0.0f, 1, 0, 1u), 0, 0, 7u);
    const float e11 = take(take(take(take(0.0f, 1, 1, 0u), 1, 0, 2u), 0, 1, 6u), 0, 0, 8u);
    const int ih = 2 * a, iw = 2 * b;
    T* o = gx + (nc * g.H + ih) * (size_t)g.W + iw;
    if ((g.W & 1) == 0) {
        // even rows: the two columns of the block are one aligned pair
        auto store2 = [](T* p, float v0, float v1) {
            if constexpr (sizeof(T) == 4) {
                *reinterpret_cast<float2*>(p) = make_float2(v0, v1);
            } else {
                *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(v0, v1);
            }
        };
        store2(o, e00, e01);
        if (ih + 1 < g.H) store2(o + g.W, e10, e11);
        return;
    }
    const bool right = iw + 1 < g.W;
    o[0] = from_f32<T>(e00);
    if (right) o[1] = from_f32<T>(e01);
    if (ih + 1 < g.H) {
        o[g.W] = from_f32<T>(e10);
        if (right) o[g.W + 1] = from_f32<T>(e11);
    }
}

// ---------------------------------------------------------------------------------- grad_x
// Gather form: one thread per input element visits, in ascending tap order, the outputs that read
// it, and takes coef * grad_y from those whose winner is that tap.  No atomics, fixed order.
// BR: 0 both branches, 1 min branch only, 2 max branch only.
// ST: 0 = strides from the descriptor, 2 = both strides are 2 (shifts instead of divisions).
template <typename T, int BR, int ST>
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
        if (nh < 0 || (ST == 2 ? (nh & 1) : nh % g.sh) != 0) continue;
        const int oh = ST == 2 ? nh >> 1 : nh / g.sh;
        if (oh >= g.OH) continue;
        for (int s = 0; s < g.S; ++s) {
            const int nw = iw + g.pw - s * g.dw;
            if (nw < 0 || (ST == 2 ? (nw & 1) : nw % g.sw) != 0) continue;
            const int ow = ST == 2 ? nw >> 1 : nw / g.sw;
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

// grad_x for 3x3 windows, stride 1, dilation 1: a thread owns a strip of 4 input columns x RT
// input rows and slides a window of three rows of (grad_y, winner code) down it.  Input (ih, iw)
// is read by output (ih + ph - r, iw + pw - s) through tap (r, s); the contributions are taken in
// ascending tap order.  Outputs outside the plane load as gradient 0.
template <int L, bool VEC>
__device__ __forceinline__ void dw_load_codes(const uint8_t* rp, bool row_ok, unsigned mask, unsigned* out) {
    if (!row_ok) mask = 0;
    if constexpr (VEC) {
        out[0] = (mask & 1u) ? __ldg(rp) : 0u;
#pragma unroll
        for (int i = 1; i + 4 <= L; i += 4) {
            const unsigned v = ((mask >> i) & 1u) ? __ldg(reinterpret_cast<const unsigned*>(rp + i)) : 0u;
            out[i] = v & 0xffu; out[i + 1] = (v >> 8) & 0xffu; out[i + 2] = (v >> 16) & 0xffu; out[i + 3] = v >> 24;
        }
#pragma unroll
        for (int i = 1 + ((L - 1) / 4) * 4; i < L; ++i) out[i] = ((mask >> i) & 1u) ? __ldg(rp + i) : 0u;
    } else {
#pragma unroll
        for (int i = 0; i < L; ++i) out[i] = ((mask >> i) & 1u) ? __ldg(rp + i) : 0u;
    }
}

template <typename T, int BR, bool VEC>
__global__ void __launch_bounds__(256)
dw_bwd_gx3_kernel(Geo g, const float* __restrict__ alpha, const float* __restrict__ beta,
                  const T* __restrict__ gy, const uint8_t* __restrict__ codes, T* __restrict__ gx,
                  int QPR, int strips, unsigned total) {
    constexpr int RT = 6, L = 6;
    const unsigned q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= total) return;
    const unsigned t = q / (unsigned)QPR;
    const int qx = (int)(q - t * (unsigned)QPR);
    const size_t nc = t / (unsigned)strips;
    const int ih0 = (int)(t - (unsigned)nc * (unsigned)strips) * RT;
    const int c = (int)((unsigned)nc % (unsigned)g.C);
    const int iw0 = qx * 4;
    const float a = (BR == 0 && alpha) ? alpha[c] : 1.0f, b = (BR == 0 && beta) ? beta[c] : 1.0f;
    const T* gp = gy + nc * (size_t)g.OH * g.OW;
    const uint8_t* cp = codes + nc * (size_t)g.OH * g.OW;
    const int ob = ih0 + g.ph - 2, c0 = iw0 + g.pw - 2;   // first output row / column of the window
    const bool full = (iw0 + 3 < g.W) && ((g.W & 3) == 0);
    T gw_[3][L];
    unsigned cw[3][L];
    const unsigned cmask = dw_col_mask(c0, L, g.OW);
    const T* grp0 = gp + (ptrdiff_t)ob * g.OW + c0;
    const uint8_t* crp0 = cp + (ptrdiff_t)ob * g.OW + c0;
    auto load = [&](int rho) {
        const int oh = ob + rho;
        const bool ok = oh >= 0 && oh < g.OH;
        dw_load_row<T, L, VEC>(grp0 + rho * g.OW, ok, cmask, gw_[rho % 3]);
        dw_load_codes<L, VEC>(crp0 + rho * g.OW, ok, cmask, cw[rho % 3]);
    };
    load(0);
    load(1);
#pragma unroll
    for (int k = 0; k < RT; ++k) {
        if (ih0 + k >= g.H) break;
        load(k + 2);
        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int r = 0; r < 3; ++r)
#pragma unroll
            for (int sx = 0; sx < 3; ++sx)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const unsigned code = cw[(k + 2 - r) % 3][j + 2 - sx];
                    const float gv = to_f32(gw_[(k + 2 - r) % 3][j + 2 - sx]);
                    const unsigned tap = (unsigned)(r * 3 + sx);
                    if ((BR == 0 || BR == 1) && (code & 15u) == tap) acc[j] = (BR == 0) ? __fmaf_rn(a, gv, acc[j]) : acc[j] + gv;
                    if ((BR == 0 || BR == 2) && (code >> 4) == tap) acc[j] = (BR == 0) ? __fmaf_rn(b, gv, acc[j]) : acc[j] + gv;
                }
        const size_t o = (nc * g.H + ih0 + k) * (size_t)g.W + iw0;
        if (full) {
            if constexpr (sizeof(T) == 4) {
                *reinterpret_cast<float4*>(gx + o) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            } else {
                const __nv_bfloat162 p01 = __floats2bfloat162_rn(acc[0], acc[1]);
                const __nv_bfloat162 p23 = __floats2bfloat162_rn(acc[2], acc[3]);
                *reinterpret_cast<uint2*>(gx + o) = make_uint2(*reinterpret_cast<const unsigned*>(&p01),
                                                               *reinterpret_cast<const unsigned*>(&p23));
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (iw0 + j < g.W) gx[o + j] = from_f32<T>(acc[j]);
        }
    }
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
    __shared__ float wsm[2][16];     // the channel's weights (min branch / max branch) as fp32
    const int c = blockIdx.x, chunk = blockIdx.y, tid = threadIdx.x;
    for (int e = tid; e < kDwAcc * 256; e += 256) col[e] = 0.0f;
    if (tid < 32) {
        const int br = tid >> 4, tp = tid & 15;
        const T* src = (br == 1 && PAR) ? w2 : w;
        wsm[br][tp] = tp < g.RS ? to_f32(__ldg(src + (size_t)c * g.RS + tp)) : 0.0f;
    }
    __syncthreads();
    const unsigned plane = (unsigned)g.OH * g.OW;
    const unsigned items = (unsigned)g.N * plane;
    const unsigned per = (items + nchunks - 1) / nchunks;
    const unsigned lo = min(items, (unsigned)chunk * per), hi = min(items, lo + per);
    float* mine = col + tid;
    float sa = 0.0f, sb = 0.0f, ss = 0.0f;   // sum g * min value, sum g * max value, sum g
    constexpr int U = 4;                      // items in flight per thread: every load of a batch is issued first
    for (unsigned it0 = lo + tid; it0 < hi; it0 += 256 * U) {
        float gv[U];
        unsigned code[U];
        T xa[U], xb[U];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned it = it0 + u * 256;
            ok[u] = it < hi;
            const unsigned n = it / plane;
            const unsigned pix = it - n * plane;
            const size_t o = ((size_t)n * g.C + c) * plane + pix;
            gv[u] = ok[u] ? to_f32(__ldg(gy + o)) : 0.0f;
            code[u] = ok[u] ? (unsigned)__ldg(codes + o) : 0u;
        }
        if (need_ab) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const unsigned it = it0 + u * 256;
                const unsigned n = it / plane;
                const unsigned pix = it - n * plane;
                const int oh = (int)(pix / (unsigned)g.OW), ow = (int)(pix - (unsigned)oh * (unsigned)g.OW);
                const T* xp = x + ((size_t)n * g.C + c) * (size_t)g.H * g.W;
                xa[u] = xb[u] = zero_of<T>();
                if (BR == 0 || BR == 1) {
                    const unsigned tp = code[u] & 15u;
                    const int ih = oh * g.sh - g.ph + (int)(tp / g.S) * g.dh, iw = ow * g.sw - g.pw + (int)(tp % g.S) * g.dw;
                    if (ok[u] && ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) xa[u] = __ldg(xp + (size_t)ih * g.W + iw);
                }
                if (BR == 0 || BR == 2) {
                    const unsigned tp = code[u] >> 4;
                    const int ih = oh * g.sh - g.ph + (int)(tp / g.S) * g.dh, iw = ow * g.sw - g.pw + (int)(tp % g.S) * g.dw;
                    if (ok[u] && ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) xb[u] = __ldg(xp + (size_t)ih * g.W + iw);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (!ok[u]) continue;
            ss += gv[u];
            if (BR == 0 || BR == 1) {
                const unsigned tp = code[u] & 15u;
                mine[tp * 256] += gv[u];
                if (need_ab) sa = __fmaf_rn(gv[u], tap_add(xa[u], from_f32<T>(wsm[0][tp])), sa);
            }
            if (BR == 0 || BR == 2) {
                const unsigned tp = code[u] >> 4;
                mine[(16 + tp) * 256] += gv[u];
                if (need_ab) sb = __fmaf_rn(gv[u], tap_add(xb[u], from_f32<T>(wsm[1][tp])), sb);
            }
        }
    }
    mine[(2 * 16) * 256] = sa;
    mine[(2 * 16 + 1) * 256] = sb;
    mine[(2 * 16 + 2) * 256] = ss;
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

// Parameter gradients for 3x3 windows, dilation 1, stride SW: the same strips and register window
// as the forward.  The branch values of grad_alpha / grad_beta are the extrema recomputed from the
// window (no gathers); the per-tap sums take the winners from the codes.  CTA (c, chunk) walks the
// strips of its images; accumulators and reduction as in dw_bwd_params_kernel.
template <typename T, int BR, bool PAR, int SW, bool VEC>
__global__ void __launch_bounds__(256)
dw_bwd_params3_kernel(Geo g, const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ w2,
                      const T* __restrict__ gy, const uint8_t* __restrict__ codes,
                      float* __restrict__ partial, int nchunks, int need_ab, int QPR, int strips) {
    constexpr int RT = kDwRT;
    constexpr int L = 3 * SW + 3;
    constexpr bool PACKED = sizeof(T) == 2 && SW == 1;
    extern __shared__ float col[];   // [kDwAcc][256]
    const int c = blockIdx.x, chunk = blockIdx.y, tid = threadIdx.x;
    for (int e = tid; e < kDwAcc * 256; e += 256) col[e] = 0.0f;
    __syncthreads();
    T wa[9], wb[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) {
        wa[i] = __ldg(w + (size_t)c * 9 + i);
        wb[i] = PAR ? __ldg(w2 + (size_t)c * 9 + i) : wa[i];
    }
    const int per = (g.N + nchunks - 1) / nchunks;
    const int n_lo = min(g.N, chunk * per), n_hi = min(g.N, n_lo + per);
    const unsigned sq = (unsigned)strips * QPR;                 // strips x quads of one plane
    const unsigned nitems = (unsigned)(n_hi - n_lo) * sq;
    const size_t plane = (size_t)g.OH * g.OW;
    float* mine = col + tid;
    float sa = 0.0f, sb = 0.0f, ss = 0.0f;
    for (unsigned it = tid; it < nitems; it += 256) {
        const unsigned nl = it / sq;
        const unsigned rem = it - nl * sq;
        const int st = (int)(rem / (unsigned)QPR), qx = (int)(rem - (unsigned)st * QPR);
        const size_t nc = (size_t)(n_lo + nl) * g.C + c;
        const int oh0 = st * RT, ow0 = qx * 4;
        const T* gp = gy + nc * plane + ow0;
        const uint8_t* cp = codes + nc * plane + ow0;
        const bool full = (ow0 + 3 < g.OW) && ((g.OW & 3) == 0);
        const int ih0 = oh0 * SW - g.ph, c0 = ow0 * SW - g.pw;
        T win[3][L];
        const unsigned cmask = need_ab ? dw_col_mask(c0, L, g.W) : 0u;
        const T* rp0 = x + nc * (size_t)g.H * g.W + (ptrdiff_t)ih0 * g.W + c0;
        auto load = [&](int rho) {
            const int ih = ih0 + rho;
            dw_load_row<T, L, VEC>(rp0 + rho * g.W, need_ab && ih >= 0 && ih < g.H, cmask, win[rho % 3]);
        };
        load(0);
        load(1);
#pragma unroll
        for (int k = 0; k < RT; ++k) {
            const int oh = oh0 + k;
            if (oh >= g.OH) break;
#pragma unroll
            for (int rho = (k == 0 ? 2 : (k - 1) * SW + 3); rho <= k * SW + 2; ++rho) load(rho);
            float gq[4];
            unsigned cq;
            if (full) {
                T tmp[4];
                load4(gp + (size_t)oh * g.OW, tmp);
#pragma unroll
                for (int j = 0; j < 4; ++j) gq[j] = to_f32(tmp[j]);
                cq = __ldg(reinterpret_cast<const unsigned*>(cp + (size_t)oh * g.OW));
            } else {
                cq = 0u;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool ok = ow0 + j < g.OW;
                    gq[j] = ok ? to_f32(__ldg(gp + (size_t)oh * g.OW + j)) : 0.0f;
                    if (ok) cq |= (unsigned)__ldg(cp + (size_t)oh * g.OW + j) << (8 * j);
                }
            }
            // bf16 at stride 1: the branch values of the four outputs on packed pairs, as in the forward
            float bmn[4] = {0.0f, 0.0f, 0.0f, 0.0f}, bmx[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if constexpr (PACKED) {
                if (need_ab) {
#pragma unroll
                    for (int pr = 0; pr < 2; ++pr) {
                        unsigned ta[9], tb[PAR ? 9 : 1];
#pragma unroll
                        for (int tap = 0; tap < 9; ++tap) {
                            const T* row = win[(k + tap / 3) % 3];
                            const int i = 2 * pr + tap % 3;
                            const unsigned xv = (unsigned)__bfloat16_as_ushort(row[i]) |
                                                ((unsigned)__bfloat16_as_ushort(row[i + 1]) << 16);
                            ta[tap] = dw_hadd2(xv, 0x00010001u * (unsigned)__bfloat16_as_ushort(wa[tap]));
                            if constexpr (PAR) tb[tap] = dw_hadd2(xv, 0x00010001u * (unsigned)__bfloat16_as_ushort(wb[tap]));
                        }
                        const unsigned* tm = PAR ? tb : ta;
                        if (BR == 0 || BR == 1) {
                            const unsigned m2 = dw_fold9_h2(ta, true);
                            bmn[2 * pr] = __uint_as_float(m2 << 16);
                            bmn[2 * pr + 1] = __uint_as_float(m2 & 0xffff0000u);
                        }
                        if (BR == 0 || BR == 2) {
                            const unsigned m2 = dw_fold9_h2(tm, false);
                            bmx[2 * pr] = __uint_as_float(m2 << 16);
                            bmx[2 * pr + 1] = __uint_as_float(m2 & 0xffff0000u);
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (!full && ow0 + j >= g.OW) continue;
                const float gv = gq[j];
                const unsigned code = (cq >> (8 * j)) & 0xffu;
                ss += gv;
                if (BR == 0 || BR == 1) mine[(code & 15u) * 256] += gv;
                if (BR == 0 || BR == 2) mine[(16 + (code >> 4)) * 256] += gv;
                if (need_ab) {
                    if constexpr (PACKED) {
                        if (BR == 0 || BR == 1) sa = __fmaf_rn(gv, bmn[j], sa);
                        if (BR == 0 || BR == 2) sb = __fmaf_rn(gv, bmx[j], sb);
                    } else {
                        float ta[9], tb[PAR ? 9 : 1];
#pragma unroll
                        for (int tap = 0; tap < 9; ++tap) {
                            const T xv = win[(k * SW + tap / 3) % 3][j * SW + tap % 3];
                            ta[tap] = tap_add(xv, wa[tap]);
                            if constexpr (PAR) tb[tap] = tap_add(xv, wb[tap]);
                        }
                        const float* tm = PAR ? tb : ta;
                        if (BR == 0 || BR == 1) sa = __fmaf_rn(gv, dw_fold9(ta, true), sa);
                        if (BR == 0 || BR == 2) sb = __fmaf_rn(gv, dw_fold9(tm, false), sb);
                    }
                }
            }
        }
    }
    mine[(2 * 16) * 256] = sa;
    mine[(2 * 16 + 1) * 256] = sb;
    mine[(2 * 16 + 2) * 256] = ss;
    __syncthreads();
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

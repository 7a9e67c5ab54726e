// One-dimensional tropical convolution with long windows (Section 3.2; the paper's audio networks
// open with a window of 80 samples at stride 4 on signals of 16000 samples, one input channel).
// The layers arrive through the three-dimensional entry points as 1 x 1 x S windows on signals of
// unit depth and height, and use the winner layouts of those entry points.
//
// Forward: the signal segment of a block sits in shared memory split by phase (index modulo the
// stride), so that the taps s = q * stride + p of neighbouring output positions read neighbouring
// words; a lane owns four consecutive positions and a few output channels, and walks the window
// with a register window of eight samples per phase.  Taps beyond S hold NaN weights, which
// min / max skip.  Backward: grad_x by scattering into block-private shared-memory arrays (threads
// of even and odd index own one array each, a thread's positions cannot reach past its neighbour's),
// the parameter gradients by private per-thread columns per tap; every sum has a fixed order.
#pragma once
#include <type_traits>

#include "tconv_3d.cuh"

namespace tconv {

constexpr int kF1Threads = 128;  // four warps: one tile of positions, four groups of output channels
constexpr int kF1Pos = 128;      // output positions per block: four per lane
constexpr int kGx1Threads = 64;  // most threads of a grad_x block

template <typename T, int N>
struct alignas(sizeof(T) * N > 16 ? 16 : sizeof(T) * N) Vec {
    T v[N];
};

__device__ __forceinline__ float fmin3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// packed bf16 pairs (two adjacent output positions per register)
__device__ __forceinline__ unsigned h1_add2(unsigned a, unsigned b) {
    unsigned d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ unsigned h1_min2(unsigned a, unsigned b) {
    unsigned d;
    asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ unsigned h1_max2(unsigned a, unsigned b) {
    unsigned d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// {w, w} of a weight in the layer's type (bf16 only; the fp32 overload is never called)
__device__ __forceinline__ unsigned h1_dup(__nv_bfloat16 v) { return 0x00010001u * (unsigned)__bfloat16_as_ushort(v); }
__device__ __forceinline__ unsigned h1_dup(float) { return 0u; }

template <typename T> __device__ __forceinline__ T nan_of();
template <> __device__ __forceinline__ float nan_of<float>() { return __int_as_float(0x7fc00000); }
template <> __device__ __forceinline__ __nv_bfloat16 nan_of<__nv_bfloat16>() {
    return __ushort_as_bfloat16((unsigned short)0x7fc0);
}

// Branches of a layer: 0 min only, 1 max only, 2 both on one weight (compound), 3 both on two
// weights (parallel).
__host__ __device__ constexpr bool has_min(int br) { return br != 1; }
__host__ __device__ constexpr bool has_max(int br) { return br != 0; }
// Output channels per thread: eight while one extremum per output is live, else four.
__host__ __device__ constexpr int f1_kt(int br, bool win) { return (br >= 2 || win) ? 4 : 8; }

// Row pitch of the staged signal segment: the window of the last lane ends at 4 * 31 + q4 + 3.
__host__ __device__ constexpr int f1_xw(int q4) { return (kF1Pos + q4 + 4 + 7) & ~7; }

// Forward.  grid (ceil(OL / 128), ceil(K / (4 * KT)), N), 128 threads.  Shared memory: the block's
// signal segment of one input channel by phase, xs[ST][xw] with xs[p][i] = x[(P0 + i) * ST + p - pad]
// (zero outside the signal), xw = 128 + q4 + 4 rounded up to a multiple of eight, and the weights
// of that channel for the block's 4 * KT output channels, ws[s][4 * KT] for s < q4 * ST (NaN for
// s >= S; bf16 layers keep them as 4-byte {w, w} pairs), twice in parallel mode.  q4 = ceil(S / ST)
// rounded up to a multiple of four.  WIN: a second copy of the weights by output channel follows,
// wst[4 * KT][q4 * ST] in the layer's type (twice in parallel mode).
template <typename T, int ST, int BR, bool WIN>
__global__ void __launch_bounds__(kF1Threads)
fwd1d_kernel(Geo3 g, int q4, const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ w2,
             const float* __restrict__ alpha, const float* __restrict__ beta,
             const float* __restrict__ bias, T* __restrict__ y, void* __restrict__ winners) {
    constexpr int KT = f1_kt(BR, WIN);
    constexpr int KB = 4 * KT;
    constexpr bool MIN = has_min(BR), MAX = has_max(BR);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int xw = f1_xw(q4);
    // bf16: two adjacent positions per register, the weights staged as {w, w} pairs
    constexpr bool PK = sizeof(T) == 2;
    using WT = typename std::conditional<PK, unsigned, T>::type;
    T* xs = reinterpret_cast<T*>(smem_raw);
    WT* wsw = reinterpret_cast<WT*>(xs + ST * xw);
    WT* wsw2 = wsw + q4 * ST * KB;
    T* ws = reinterpret_cast<T*>(wsw);      // (the views used by the unpacked paths)
    T* ws2 = reinterpret_cast<T*>(wsw2);
    // WIN: a second copy of the weights by output channel, wst[kk][s], for the second step
    T* wst = reinterpret_cast<T*>(wsw2 + (BR == 3 ? q4 * ST * KB : 0));
    T* wst2 = wst + q4 * ST * KB;
    const int tid = threadIdx.x, lane = tid & 31, wv = tid >> 5;
    const int P0 = blockIdx.x * kF1Pos, n = blockIdx.z;
    const int kb0 = blockIdx.y * KB, k0 = kb0 + wv * KT;
    const int L = g.W, OL = g.OW, S = g.S;
    float out[KT][4];
    int win[KT][4];
#pragma unroll
    for (int kk = 0; kk < KT; ++kk)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            out[kk][j] = (g.chan == CH_SUM) ? 0.0f : (g.chan == CH_MAX ? -INFINITY : INFINITY);
            win[kk][j] = -1;
        }
    for (int c = 0; c < g.C; ++c) {
        __syncthreads();
        {   // stage the signal segment by phase and the weights by tap
            const T* xc = x + ((size_t)n * g.C + c) * L;
            const long long base = (long long)P0 * ST - g.pw;
            for (int j = tid; j < xw * ST; j += kF1Threads) {
                const long long gi = base + j;
                xs[(j % ST) * xw + j / ST] = (gi >= 0 && gi < L) ? xc[gi] : zero_of<T>();
            }
            const int span = q4 * ST;
            for (int i = tid; i < KB * span; i += kF1Threads) {
                const int kk = i / span, s = i - kk * span, k = kb0 + kk;
                T a = zero_of<T>(), b = zero_of<T>();
                if (s >= S) a = b = nan_of<T>();
                else if (k < g.K) {
                    const size_t wi = ((size_t)k * g.C + c) * S + s;
                    a = w[wi];
                    if (BR == 3) b = w2[wi];
                }
                if constexpr (PK) {
                    wsw[s * KB + kk] = h1_dup(a);
                    if (BR == 3) wsw2[s * KB + kk] = h1_dup(b);
                } else {
                    ws[s * KB + kk] = a;
                    if (BR == 3) ws2[s * KB + kk] = b;
                }
                if constexpr (WIN) {
                    wst[i] = a;
                    if (BR == 3) wst2[i] = b;
                }
            }
        }
        __syncthreads();
        float mn[KT][4], mx[KT][4];
        int amn[KT][4], amx[KT][4];
#pragma unroll
        for (int kk = 0; kk < KT; ++kk)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                mn[kk][j] = INFINITY; mx[kk][j] = -INFINITY; amn[kk][j] = 0; amx[kk][j] = 0;
            }
        if constexpr (PK && !WIN) {
            // positions (0, 1) and (2, 3) of the lane as pairs; a tap at an odd offset into the window
            // takes the pairs shifted by one element
            unsigned mn2[KT][2], mx2[KT][2];
#pragma unroll
            for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                for (int pr = 0; pr < 2; ++pr) { mn2[kk][pr] = 0x7f807f80u; mx2[kk][pr] = 0xff80ff80u; }
#pragma unroll
            for (int p = 0; p < ST; ++p) {
                const T* xp = xs + p * xw + 4 * lane;
                for (int q0 = 0; q0 < q4; q0 += 4) {
                    const uint2 lo = *reinterpret_cast<const uint2*>(xp + q0);
                    const uint2 hi = *reinterpret_cast<const uint2*>(xp + q0 + 4);
                    const unsigned ev[4] = {lo.x, lo.y, hi.x, hi.y};
                    const unsigned od[3] = {__byte_perm(lo.x, lo.y, 0x5432), __byte_perm(lo.y, hi.x, 0x5432),
                                            __byte_perm(hi.x, hi.y, 0x5432)};
#pragma unroll
                    for (int dq = 0; dq < 4; dq += 2) {
                        const int s0 = (q0 + dq) * ST + p, s1 = s0 + ST;
                        const Vec<unsigned, KT> wa0 = *reinterpret_cast<const Vec<unsigned, KT>*>(wsw + s0 * KB + wv * KT);
                        const Vec<unsigned, KT> wa1 = *reinterpret_cast<const Vec<unsigned, KT>*>(wsw + s1 * KB + wv * KT);
                        Vec<unsigned, KT> wb0 = wa0, wb1 = wa1;
                        if constexpr (BR == 3) {
                            wb0 = *reinterpret_cast<const Vec<unsigned, KT>*>(wsw2 + s0 * KB + wv * KT);
                            wb1 = *reinterpret_cast<const Vec<unsigned, KT>*>(wsw2 + s1 * KB + wv * KT);
                        }
#pragma unroll
                        for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                            for (int pr = 0; pr < 2; ++pr) {
                                const unsigned x0 = ev[dq / 2 + pr], x1 = od[dq / 2 + pr];
                                const unsigned t0 = h1_add2(x0, wa0.v[kk]), t1 = h1_add2(x1, wa1.v[kk]);
                                if constexpr (MIN) mn2[kk][pr] = h1_min2(h1_min2(mn2[kk][pr], t0), t1);
                                if constexpr (BR == 3) {
                                    const unsigned u0 = h1_add2(x0, wb0.v[kk]), u1 = h1_add2(x1, wb1.v[kk]);
                                    mx2[kk][pr] = h1_max2(h1_max2(mx2[kk][pr], u0), u1);
                                } else if constexpr (MAX) {
                                    mx2[kk][pr] = h1_max2(h1_max2(mx2[kk][pr], t0), t1);
                                }
                            }
                    }
                }
            }
#pragma unroll
            for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                for (int pr = 0; pr < 2; ++pr) {
                    mn[kk][2 * pr] = __uint_as_float(mn2[kk][pr] << 16);
                    mn[kk][2 * pr + 1] = __uint_as_float(mn2[kk][pr] & 0xffff0000u);
                    mx[kk][2 * pr] = __uint_as_float(mx2[kk][pr] << 16);
                    mx[kk][2 * pr + 1] = __uint_as_float(mx2[kk][pr] & 0xffff0000u);
                }
        } else if constexpr (!WIN) {
#pragma unroll
            for (int p = 0; p < ST; ++p) {
                const T* xp = xs + p * xw + 4 * lane;
                for (int q0 = 0; q0 < q4; q0 += 4) {
                    T r[8];
                    *reinterpret_cast<Vec<T, 4>*>(r) = *reinterpret_cast<const Vec<T, 4>*>(xp + q0);
                    *reinterpret_cast<Vec<T, 4>*>(r + 4) = *reinterpret_cast<const Vec<T, 4>*>(xp + q0 + 4);
#pragma unroll
                    for (int dq = 0; dq < 4; dq += 2) {
                        const int s0 = (q0 + dq) * ST + p, s1 = s0 + ST;
                        const Vec<T, KT> wa0 = *reinterpret_cast<const Vec<T, KT>*>(ws + s0 * KB + wv * KT);
                        const Vec<T, KT> wa1 = *reinterpret_cast<const Vec<T, KT>*>(ws + s1 * KB + wv * KT);
                        Vec<T, KT> wb0 = wa0, wb1 = wa1;
                        if constexpr (BR == 3) {
                            wb0 = *reinterpret_cast<const Vec<T, KT>*>(ws2 + s0 * KB + wv * KT);
                            wb1 = *reinterpret_cast<const Vec<T, KT>*>(ws2 + s1 * KB + wv * KT);
                        }
#pragma unroll
                        for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float t0 = tap_add(r[dq + j], wa0.v[kk]);
                                const float t1 = tap_add(r[dq + 1 + j], wa1.v[kk]);
                                if constexpr (MIN) mn[kk][j] = fmin3(mn[kk][j], t0, t1);
                                if constexpr (BR == 3) {
                                    const float u0 = tap_add(r[dq + j], wb0.v[kk]);
                                    const float u1 = tap_add(r[dq + 1 + j], wb1.v[kk]);
                                    mx[kk][j] = fmax3(mx[kk][j], u0, u1);
                                } else if constexpr (MAX) {
                                    mx[kk][j] = fmax3(mx[kk][j], t0, t1);
                                }
                            }
                    }
                }
            }
        } else {
            // Winners in two steps.  First the windows are walked in blocks of BQ q (BQ * ST = 4 or
            // 8 consecutive taps, blocks ascending): a block's extremum replaces the running one only
            // when it is strictly better, and the block is remembered.  Then, per output and branch,
            // the taps of the remembered block are formed again, highest first, and the lowest one
            // that equals the extremum is the winner.
            constexpr int BQ = ST == 4 ? 2 : 4;
            const T* xl = xs + 4 * lane;
            int bmn[KT][4], bmx[KT][4];
#pragma unroll
            for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                for (int j = 0; j < 4; ++j) bmn[kk][j] = bmx[kk][j] = 0;
            if constexpr (PK) {
                // bf16: the first step on pairs of positions; per half a mask says where the block is
                // strictly better, and takes the block's first q into that half of the block register
                unsigned mn2[KT][2], mx2[KT][2], bmn2[KT][2], bmx2[KT][2];
#pragma unroll
                for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                    for (int pr = 0; pr < 2; ++pr) {
                        mn2[kk][pr] = 0x7f807f80u; mx2[kk][pr] = 0xff80ff80u; bmn2[kk][pr] = bmx2[kk][pr] = 0u;
                    }
                for (int q0 = 0; q0 < q4; q0 += 4) {
                    unsigned ev[ST][4], od[ST][3];
#pragma unroll
                    for (int p = 0; p < ST; ++p) {
                        const uint2 lo = *reinterpret_cast<const uint2*>(xl + p * xw + q0);
                        const uint2 hi = *reinterpret_cast<const uint2*>(xl + p * xw + q0 + 4);
                        ev[p][0] = lo.x; ev[p][1] = lo.y; ev[p][2] = hi.x; ev[p][3] = hi.y;
                        od[p][0] = __byte_perm(lo.x, lo.y, 0x5432);
                        od[p][1] = __byte_perm(lo.y, hi.x, 0x5432);
                        od[p][2] = __byte_perm(hi.x, hi.y, 0x5432);
                    }
                    unsigned cm2[KT][2], cx2[KT][2];
#pragma unroll
                    for (int dq = 0; dq < 4; dq += 2) {
                        if (dq % BQ == 0) {
#pragma unroll
                            for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                                for (int pr = 0; pr < 2; ++pr) { cm2[kk][pr] = 0x7f807f80u; cx2[kk][pr] = 0xff80ff80u; }
                        }
#pragma unroll
                        for (int p = 0; p < ST; ++p) {
                            const int s0 = (q0 + dq) * ST + p, s1 = s0 + ST;
                            const Vec<unsigned, KT> wa0 = *reinterpret_cast<const Vec<unsigned, KT>*>(wsw + s0 * KB + wv * KT);
                            const Vec<unsigned, KT> wa1 = *reinterpret_cast<const Vec<unsigned, KT>*>(wsw + s1 * KB + wv * KT);
                            Vec<unsigned, KT> wb0 = wa0, wb1 = wa1;
                            if constexpr (BR == 3) {
                                wb0 = *reinterpret_cast<const Vec<unsigned, KT>*>(wsw2 + s0 * KB + wv * KT);
                                wb1 = *reinterpret_cast<const Vec<unsigned, KT>*>(wsw2 + s1 * KB + wv * KT);
                            }
#pragma unroll
                            for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                                for (int pr = 0; pr < 2; ++pr) {
                                    const unsigned x0 = ev[p][dq / 2 + pr], x1 = od[p][dq / 2 + pr];
                                    const unsigned t0 = h1_add2(x0, wa0.v[kk]), t1 = h1_add2(x1, wa1.v[kk]);
                                    if constexpr (MIN) cm2[kk][pr] = h1_min2(h1_min2(cm2[kk][pr], t0), t1);
                                    if constexpr (BR == 3) {
                                        const unsigned u0 = h1_add2(x0, wb0.v[kk]), u1 = h1_add2(x1, wb1.v[kk]);
                                        cx2[kk][pr] = h1_max2(h1_max2(cx2[kk][pr], u0), u1);
                                    } else if constexpr (MAX) {
                                        cx2[kk][pr] = h1_max2(h1_max2(cx2[kk][pr], t0), t1);
                                    }
                                }
                        }
                        if ((dq + 2) % BQ == 0) {
                            const unsigned qb2 = 0x00010001u * (unsigned)(q0 + dq + 2 - BQ);
#pragma unroll
                            for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                                for (int pr = 0; pr < 2; ++pr) {
                                    if constexpr (MIN) {
                                        const unsigned m = __hlt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&cm2[kk][pr]),
                                                                       *reinterpret_cast<const __nv_bfloat162*>(&mn2[kk][pr]));
                                        mn2[kk][pr] = h1_min2(mn2[kk][pr], cm2[kk][pr]);
                                        bmn2[kk][pr] = (qb2 & m) | (bmn2[kk][pr] & ~m);
                                    }
                                    if constexpr (MAX) {
                                        const unsigned m = __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&cx2[kk][pr]),
                                                                       *reinterpret_cast<const __nv_bfloat162*>(&mx2[kk][pr]));
                                        mx2[kk][pr] = h1_max2(mx2[kk][pr], cx2[kk][pr]);
                                        bmx2[kk][pr] = (qb2 & m) | (bmx2[kk][pr] & ~m);
                                    }
                                }
                        }
                    }
                }
#pragma unroll
                for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                    for (int pr = 0; pr < 2; ++pr) {
                        mn[kk][2 * pr] = __uint_as_float(mn2[kk][pr] << 16);
                        mn[kk][2 * pr + 1] = __uint_as_float(mn2[kk][pr] & 0xffff0000u);
                        mx[kk][2 * pr] = __uint_as_float(mx2[kk][pr] << 16);
                        mx[kk][2 * pr + 1] = __uint_as_float(mx2[kk][pr] & 0xffff0000u);
                        bmn[kk][2 * pr] = (int)(bmn2[kk][pr] & 0xffffu);
                        bmn[kk][2 * pr + 1] = (int)(bmn2[kk][pr] >> 16);
                        bmx[kk][2 * pr] = (int)(bmx2[kk][pr] & 0xffffu);
                        bmx[kk][2 * pr + 1] = (int)(bmx2[kk][pr] >> 16);
                    }
            } else
            for (int q0 = 0; q0 < q4; q0 += 4) {
                T r[ST][8];
#pragma unroll
                for (int p = 0; p < ST; ++p) {
                    *reinterpret_cast<Vec<T, 4>*>(r[p]) = *reinterpret_cast<const Vec<T, 4>*>(xl + p * xw + q0);
                    *reinterpret_cast<Vec<T, 4>*>(r[p] + 4) =
                        *reinterpret_cast<const Vec<T, 4>*>(xl + p * xw + q0 + 4);
                }
                float cmn[KT][4], cmx[KT][4];
#pragma unroll
                for (int dq = 0; dq < 4; dq += 2) {
                    if (dq % BQ == 0) {
#pragma unroll
                        for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                            for (int j = 0; j < 4; ++j) { cmn[kk][j] = INFINITY; cmx[kk][j] = -INFINITY; }
                    }
#pragma unroll
                    for (int p = 0; p < ST; ++p) {
                        const int s0 = (q0 + dq) * ST + p, s1 = s0 + ST;
                        const Vec<T, KT> wa0 = *reinterpret_cast<const Vec<T, KT>*>(ws + s0 * KB + wv * KT);
                        const Vec<T, KT> wa1 = *reinterpret_cast<const Vec<T, KT>*>(ws + s1 * KB + wv * KT);
                        Vec<T, KT> wb0 = wa0, wb1 = wa1;
                        if constexpr (BR == 3) {
                            wb0 = *reinterpret_cast<const Vec<T, KT>*>(ws2 + s0 * KB + wv * KT);
                            wb1 = *reinterpret_cast<const Vec<T, KT>*>(ws2 + s1 * KB + wv * KT);
                        }
#pragma unroll
                        for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float t0 = tap_add(r[p][dq + j], wa0.v[kk]);
                                const float t1 = tap_add(r[p][dq + 1 + j], wa1.v[kk]);
                                if constexpr (MIN) cmn[kk][j] = fmin3(cmn[kk][j], t0, t1);
                                if constexpr (BR == 3) {
                                    const float u0 = tap_add(r[p][dq + j], wb0.v[kk]);
                                    const float u1 = tap_add(r[p][dq + 1 + j], wb1.v[kk]);
                                    cmx[kk][j] = fmax3(cmx[kk][j], u0, u1);
                                } else if constexpr (MAX) {
                                    cmx[kk][j] = fmax3(cmx[kk][j], t0, t1);
                                }
                            }
                    }
                    if ((dq + 2) % BQ == 0) {   // the block that starts at q0 + dq + 2 - BQ is complete
                        const int qb = q0 + dq + 2 - BQ;
#pragma unroll
                        for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if constexpr (MIN)
                                    if (cmn[kk][j] < mn[kk][j]) { mn[kk][j] = cmn[kk][j]; bmn[kk][j] = qb; }
                                if constexpr (MAX)
                                    if (cmx[kk][j] > mx[kk][j]) { mx[kk][j] = cmx[kk][j]; bmx[kk][j] = qb; }
                            }
                    }
                }
            }
            const int span = q4 * ST;
            const T* wt = wst + wv * KT * span;
            const T* wt2 = (BR == 3 ? wst2 : wst) + wv * KT * span;
#pragma unroll
            for (int kk = 0; kk < KT; ++kk)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if constexpr (MIN) {
                        const int qb = bmn[kk][j];
                        const float m = mn[kk][j];
                        int am = 0;
#pragma unroll
                        const T* wq = wt + kk * span + qb * ST;
                        const T* xq = xl + j + qb;
#pragma unroll
                        for (int i = BQ * ST - 1; i >= 0; --i) {
                            const float t = tap_add(xq[(i % ST) * xw + i / ST], wq[i]);
                            if (t == m) am = qb * ST + i;
                        }
                        amn[kk][j] = am;
                    }
                    if constexpr (MAX) {
                        const int qb = bmx[kk][j];
                        const float m = mx[kk][j];
                        int am = 0;
#pragma unroll
                        const T* wq = wt2 + kk * span + qb * ST;
                        const T* xq = xl + j + qb;
#pragma unroll
                        for (int i = BQ * ST - 1; i >= 0; --i) {
                            const float t = tap_add(xq[(i % ST) * xw + i / ST], wq[i]);
                            if (t == m) am = qb * ST + i;
                        }
                        amx[kk][j] = am;
                    }
                }
        }
        // channel combine, channels ascending
#pragma unroll
        for (int kk = 0; kk < KT; ++kk) {
            const int k = k0 + kk;
            if (k >= g.K) continue;
            float a = 1.0f, b = 1.0f;
            if (BR >= 2) {
                if (alpha) a = alpha[(size_t)k * g.C + c];
                if (beta) b = beta[(size_t)k * g.C + c];
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if constexpr (BR >= 2) {
                    out[kk][j] = __fmaf_rn(a, mn[kk][j], out[kk][j]);
                    out[kk][j] = __fmaf_rn(b, mx[kk][j], out[kk][j]);
                } else {
                    const float m = MIN ? mn[kk][j] : mx[kk][j];
                    const int am = MIN ? amn[kk][j] : amx[kk][j];
                    if (g.chan == CH_SUM) out[kk][j] = __fadd_rn(out[kk][j], m);
                    else if (g.chan == CH_MAX) { if (m > out[kk][j]) { out[kk][j] = m; win[kk][j] = c * S + am; } }
                    else { if (m < out[kk][j]) { out[kk][j] = m; win[kk][j] = c * S + am; } }
                }
                if (WIN && g.chan == CH_SUM) {
                    const int pos = P0 + 4 * lane + j;
                    if (pos < OL)
                        ((uint16_t*)winners)[(((size_t)n * g.K + k) * g.C + c) * OL + pos] =
                            (uint16_t)((MIN ? amn[kk][j] : 0) | ((MAX ? amx[kk][j] : 0) << 8));
                }
            }
        }
    }
#pragma unroll
    for (int kk = 0; kk < KT; ++kk) {
        const int k = k0 + kk;
        if (k >= g.K) continue;
        const float bv = bias ? bias[k] : 0.0f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int pos = P0 + 4 * lane + j;
            if (pos >= OL) continue;
            float v = out[kk][j];
            if (bias) v = __fadd_rn(v, bv);
            const size_t o = ((size_t)n * g.K + k) * OL + pos;
            if (y) y[o] = from_f32<T>(v);
            if (WIN && g.chan != CH_SUM) ((int32_t*)winners)[o] = win[kk][j];
        }
    }
}

// grad_x partial sums by scattering.  grid (tiles, C * ks, N), blockDim.x = tb threads; a thread owns
// pt consecutive output positions (pt * stride >= S - stride, so its windows end before the
// positions of the thread after the next begin) and adds, channels of its slice ascending and
// positions ascending, every gradient to the winner's element of the shared-memory array of its
// parity.  The block's two arrays cover span = tb * pt * stride - stride + S elements from padded
// index tile * tb * pt * stride; their sum goes to part[slice][n][c][tile][span].
template <typename T>
__global__ void __launch_bounds__(kGx1Threads)
bwd1d_gx_kernel(Geo3 g, int pt, int ks, int span, const float* __restrict__ alpha,
                const float* __restrict__ beta, const T* __restrict__ gy,
                const void* __restrict__ winners, float* __restrict__ part) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* even = reinterpret_cast<float*>(smem_raw);
    float* odd = even + span;
    const int tid = threadIdx.x, tb = blockDim.x;
    const int tile = blockIdx.x, c = blockIdx.y / ks, slice = blockIdx.y % ks, n = blockIdx.z;
    const int OL = g.OW, st = g.sw;
    const bool twob = two_branch(g.mode), codes = g.chan == CH_SUM;
    const bool use_min = g.mode != TCONV_MAX_PLUS, use_max = g.mode != TCONV_MIN_PLUS;
    for (int i = tid; i < 2 * span; i += tb) even[i] = 0.0f;
    __syncthreads();
    float* mine = (tid & 1) ? odd : even;
    const int lp0 = tid * pt, p0 = tile * tb * pt + lp0;
    const int cnt = min(pt, OL - p0);
    const int kper = (g.K + ks - 1) / ks;
    const int kend = min(g.K, (slice + 1) * kper);
    for (int k = slice * kper; k < kend; ++k) {
        float a = 1.0f, b = 1.0f;
        if (twob) {
            if (alpha) a = alpha[k * g.C + c];
            if (beta) b = beta[k * g.C + c];
        }
        // (every tensor of the layer has fewer than 2^31 elements: 32-bit offsets)
        const T* grow = gy + ((n * g.K + k) * OL + p0);
        const uint16_t* crow = (const uint16_t*)winners + (((n * g.K + k) * g.C + c) * OL + p0);
        const int32_t* irow = (const int32_t*)winners + ((n * g.K + k) * OL + p0);
        // eight positions at a time: their winners and gradients are requested together
        for (int i0 = 0; i0 < cnt; i0 += 8) {
            int amn[8], amx[8];
            float gv[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = min(i0 + u, cnt - 1);
                if (codes) {
                    const unsigned v = crow[i];
                    amn[u] = use_min ? (int)(v & 0xFFu) : -1;
                    amx[u] = use_max ? (int)(v >> 8) : -1;
                } else {
                    const int v = irow[i] - c * g.S;
                    const int tap = (v >= 0 && v < g.S) ? v : -1;
                    amn[u] = use_min ? tap : -1;
                    amx[u] = use_min ? -1 : tap;
                }
                gv[u] = to_f32(grow[i]);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (i0 + u >= cnt) break;
                float* at = mine + (lp0 + i0 + u) * st;
                if (amn[u] >= 0) at[amn[u]] = twob ? __fmaf_rn(a, gv[u], at[amn[u]]) : at[amn[u]] + gv[u];
                if (amx[u] >= 0) at[amx[u]] = twob ? __fmaf_rn(b, gv[u], at[amx[u]]) : at[amx[u]] + gv[u];
            }
        }
    }
    __syncthreads();
    float* o = part + ((((size_t)slice * g.N + n) * g.C + c) * gridDim.x + tile) * span;
    for (int i = tid; i < span; i += tb) o[i] = even[i] + odd[i];
}

// grad_x from the partial sums: one thread per input element; the tiles that cover it (at most
// two) in ascending order, slices ascending inside a tile.
template <typename T>
__global__ void __launch_bounds__(256)
bwd1d_gx_finish_kernel(Geo3 g, int tiles, int ks, int span, int tile_x, const float* __restrict__ part,
                       T* __restrict__ gx) {
    const size_t total = (size_t)g.N * g.C * g.W;
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= total) return;
    const int i = (int)(e % g.W);
    const size_t nc = e / g.W;
    const int n = (int)(nc / g.C), c = (int)(nc % g.C);
    const int u = i + g.pw;  // padded index: position * stride + tap
    const int b = u / tile_x;
    float acc = 0.0f;
    for (int t = b - 1; t <= b; ++t) {
        if (t < 0 || t >= tiles) continue;
        const int li = u - t * tile_x;
        if (li >= span) continue;
        for (int sl = 0; sl < ks; ++sl)
            acc += part[((((size_t)sl * g.N + n) * g.C + c) * tiles + t) * span + li];
    }
    gx[e] = from_f32<T>(acc);
}

// Parameter-gradient partial sums of one (k, c) over a share of the (n, position) range: grid
// (K * C, nsplit), blockDim.x = tb (a power of two).  Shared memory: per present branch a private
// column per thread and tap, col[tap][tb], then the branch weights and tb floats for the block
// sums.  Outputs: part_min / part_max [split][k*C+c][tap] (sums of grad_y over the outputs a tap
// won), part_ab [split][k*C+c][2] (sums of grad_y * branch value, two-branch layers) and, from the
// blocks of channel 0, part_bias [split][k].  (The launch bounds keep 384 threads resident per SM: the
// host sizes the splits for one round of blocks.)
template <typename T>
__global__ void __launch_bounds__(128, 3)
bwd1d_params_kernel(Geo3 g, int nsplit, const T* __restrict__ x, const T* __restrict__ w,
                    const T* __restrict__ w2, const T* __restrict__ gy, const void* __restrict__ winners,
                    float* __restrict__ part_min, float* __restrict__ part_max,
                    float* __restrict__ part_ab, float* __restrict__ part_bias) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, tb = blockDim.x;
    const int S = g.S, OL = g.OW, L = g.W;
    const int kc = blockIdx.x, k = kc / g.C, c = kc % g.C, split = blockIdx.y;
    const bool twob = two_branch(g.mode);
    const bool use_min = g.mode != TCONV_MAX_PLUS, use_max = g.mode != TCONV_MIN_PLUS;
    // S + 1 columns per present branch: column S takes the items that have no winner in the branch
    float* cmin = reinterpret_cast<float*>(smem_raw);
    float* cmax = cmin + (use_min ? (S + 1) * tb : 0);
    float* wmin_s = cmax + (use_max ? (S + 1) * tb : 0);
    float* wmax_s = wmin_s + S;
    float* red = wmax_s + S;
    for (int i = tid; i < ((use_min ? 1 : 0) + (use_max ? 1 : 0)) * (S + 1) * tb; i += tb) cmin[i] = 0.0f;
    for (int s = tid; s < S; s += tb) {
        const size_t wi = ((size_t)k * g.C + c) * S + s;
        wmin_s[s] = to_f32(w[wi]);
        wmax_s[s] = to_f32(g.mode == TCONV_PARALLEL ? w2[wi] : w[wi]);
    }
    __syncthreads();
    const int total = g.N * OL;   // (every tensor of the layer has fewer than 2^31 elements)
    const int per = (total + nsplit - 1) / nsplit;
    const int j0 = min(total, split * per), j1 = min(total, j0 + per);
    float sa = 0.0f, sb = 0.0f, sg = 0.0f;
    // Items (n, position) of this thread: j0 + tid, + tb, ...; eight at a time.  The winners and
    // gradients of the next eight are requested before the current eight are worked on; of the
    // current eight first the branch inputs are gathered, then the columns are updated in item order.
    // An item past the end reads the first item of the row (a valid address) and counts as zero.
    const bool codes = g.chan == CH_SUM;
    const int crow = g.K * g.C * OL, cbase = (k * g.C + c) * OL;  // uint16 codes [n][k][c][pos]
    const int grow = g.K * OL, gbase = k * OL;                    // grad_y, int32 winners [n][k][pos]
    const int xrow = g.C * L, xbase = c * L;
    const uint16_t* w16 = (const uint16_t*)winners;
    const int32_t* w32 = (const int32_t*)winners;
    struct Batch {
        unsigned raw[8];
        float gv[8];
        int xpl[8];   // offset of the item's input row, -1: no item
        int li0[8];   // input index of the window's first tap
    };
    int j_cur = j0 + tid;
    int n_cur = j_cur / OL, pos_cur = j_cur - n_cur * OL;
    int cofs = n_cur * crow + cbase + pos_cur, gofs = n_cur * grow + gbase + pos_cur, xofs = n_cur * xrow + xbase;
    auto fetch = [&](Batch& bt) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const bool ok = j_cur < j1;
            const int co = ok ? cofs : cbase, go = ok ? gofs : gbase;
            bt.raw[u] = codes ? (unsigned)w16[co] : (unsigned)w32[go];
            const float gv = to_f32(gy[go]);
            bt.gv[u] = ok ? gv : 0.0f;
            bt.xpl[u] = ok ? xofs : -1;
            bt.li0[u] = pos_cur * g.sw - g.pw;
            j_cur += tb;
            pos_cur += tb;
            cofs += tb;
            gofs += tb;
            if (pos_cur >= OL) {
                const int q = pos_cur / OL;
                n_cur += q;
                pos_cur -= q * OL;
                cofs += q * (crow - OL);
                gofs += q * (grow - OL);
                xofs += q * xrow;
            }
        }
    };
    auto work = [&](const Batch& bt) {
        int amn[8], amx[8];
        float vmin[8], vmax[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int tmn, tmx;
            if (codes) {
                tmn = (int)(bt.raw[u] & 0xFFu);
                tmx = (int)(bt.raw[u] >> 8);
            } else {
                const int v = (int)bt.raw[u] - c * S;
                tmn = tmx = (v >= 0 && v < S) ? v : S;
            }
            const bool ok = bt.xpl[u] >= 0;
            amn[u] = (ok && use_min) ? tmn : S;
            amx[u] = (ok && use_max) ? tmx : S;
        }
        if (twob) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const T* xc = x + max(bt.xpl[u], 0);
                const int ta = min(amn[u], S - 1), tb2 = min(amx[u], S - 1);
                const int ia = bt.li0[u] + ta, ib = bt.li0[u] + tb2;
                const T xa = (ia >= 0 && ia < L) ? xc[ia] : zero_of<T>();
                const T xb = (ib >= 0 && ib < L) ? xc[ib] : zero_of<T>();
                vmin[u] = tap_add(xa, from_f32<T>(wmin_s[ta]));
                vmax[u] = tap_add(xb, from_f32<T>(wmax_s[tb2]));
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float gv = bt.gv[u];   // zero for an item past the end
            sg += gv;
            if (use_min) cmin[amn[u] * tb + tid] += gv;
            if (use_max) cmax[amx[u] * tb + tid] += gv;
            if (twob) {
                sa = __fmaf_rn(gv, vmin[u], sa);
                sb = __fmaf_rn(gv, vmax[u], sb);
            }
        }
    };
    {
        const int batches = (j1 - j0 + 8 * tb - 1) / (8 * tb);
        Batch ba, bb;
        fetch(ba);
        for (int it = 0; it < batches; it += 2) {
            fetch(bb);
            work(ba);
            fetch(ba);
            work(bb);
        }
    }
    __syncthreads();
    for (int s = tid; s < S; s += tb) {
        float tmin = 0.0f, tmax = 0.0f;
        for (int i = 0; i < tb; ++i) {
            const int col = (i + tid) & (tb - 1);  // rotated start: the threads of a warp read different banks
            if (use_min) tmin += cmin[s * tb + col];
            if (use_max) tmax += cmax[s * tb + col];
        }
        const size_t o = ((size_t)split * g.K * g.C + kc) * S + s;
        part_min[o] = tmin;
        part_max[o] = tmax;
    }
    const float ta = block_sum(sa, red);
    const float tb_sum = block_sum(sb, red);
    const float tg = block_sum(sg, red);
    if (tid == 0) {
        float* o = part_ab + ((size_t)split * g.K * g.C + kc) * 2;
        o[0] = ta;
        o[1] = tb_sum;
        if (c == 0) part_bias[(size_t)split * g.K + k] = tg;
    }
}

}  // namespace tconv

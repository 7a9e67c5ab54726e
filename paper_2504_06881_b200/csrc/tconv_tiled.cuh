// Tiled forward kernels: the input halo tile and a repacked weight tile are staged
// in shared memory (asynchronous copies, two stages), every thread keeps a block
// of 8 output channels x Q x 4 pixels in registers and folds taps with packed
// adds (two channels per instruction) and 3-input min / max.
//
// A CTA owns TILE_K output channels x one tile of output pixels.  Pixel tiles are
// TW columns wide and TH rows high, where rows run over the flattened (n, oh)
// space, so a tile may span several images of a small feature map.
#pragma once
#include "tconv_common.cuh"

namespace tconv {

// ----------------------------------------------------------------------------------
// small device helpers
__device__ __forceinline__ float ext3(float a, float b, float c, bool is_min) {
    float d;
    if (is_min) asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    else asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float ext2(float a, float b, bool is_min) {
    return is_min ? fminf(a, b) : fmaxf(a, b);
}
// {lo, hi} = {x + wlo, x + whi}: one packed fp32 add for two output channels.
__device__ __forceinline__ void add2(float x, float wlo, float whi, float& lo, float& hi) {
    unsigned long long xx, ww, tt;
    asm("mov.b64 %0, {%1, %1};" : "=l"(xx) : "f"(x));
    asm("mov.b64 %0, {%1, %2};" : "=l"(ww) : "f"(wlo), "f"(whi));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(tt) : "l"(xx), "l"(ww));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(tt));
}
__device__ __forceinline__ void cp_async4(void* smem, const void* gmem, bool valid) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    const int n = valid ? 4 : 0;  // 0 source bytes: the destination is zero-filled
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(s), "l"(gmem), "r"(n));
}
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N));
}

// ----------------------------------------------------------------------------------
// Weight repack: w[K][C][R][S] -> wt[ktile][Cpad][RS][TILE_K] (zero padded), so that
// the weights of a channel chunk of one k-tile are one contiguous block with the
// output channel innermost (a thread reads its 8 channels with two 16-byte loads).
// alpha / beta [K][C] -> [ktile][Cpad][TILE_K]; a missing alpha / beta becomes ones.
template <typename T>
__global__ void repack_weights_kernel(int K, int C, int RS, int tile_k, int Cpad, int nkt,
                                      const T* __restrict__ w, const T* __restrict__ w2,
                                      const float* __restrict__ alpha,
                                      const float* __restrict__ beta, float* __restrict__ wt,
                                      float* __restrict__ wt2, float* __restrict__ at,
                                      float* __restrict__ bt) {
    const size_t nw = (size_t)nkt * Cpad * RS * tile_k;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nw) {
        const int kk = (int)(i % tile_k);
        const int tap = (int)((i / tile_k) % RS);
        const int c = (int)((i / ((size_t)tile_k * RS)) % Cpad);
        const int kt = (int)(i / ((size_t)tile_k * RS * Cpad));
        const int k = kt * tile_k + kk;
        const bool ok = (k < K && c < C);
        const size_t src = ((size_t)k * C + c) * RS + tap;
        wt[i] = ok ? to_f32(w[src]) : 0.0f;
        if (wt2) wt2[i] = ok ? to_f32(w2[src]) : 0.0f;
    }
    const size_t na = (size_t)nkt * Cpad * tile_k;
    if (at && i < na) {
        const int kk = (int)(i % tile_k);
        const int c = (int)((i / tile_k) % Cpad);
        const int kt = (int)(i / ((size_t)tile_k * Cpad));
        const int k = kt * tile_k + kk;
        const bool ok = (k < K && c < C);
        at[i] = ok ? (alpha ? alpha[(size_t)k * C + c] : 1.0f) : 0.0f;
        bt[i] = ok ? (beta ? beta[(size_t)k * C + c] : 1.0f) : 0.0f;
    }
}

// ----------------------------------------------------------------------------------
struct TiledParams {
    Geo g;
    const void* x;
    const float* wt;   // repacked weights (min branch / the only weights)
    const float* wt2;  // repacked max-branch weights (parallel)
    const float* at;   // repacked alpha, beta
    const float* bt;
    const float* bias;
    void* y;
    void* winners;
    int TW, QPR, TH;   // tile: output columns, quads per row, rows of the flattened (n, oh) space
    int n_col_tiles, n_row_tiles;
    int total_rows;    // N * OH
    int NSLOTS, XW, XP;  // staged input rows per tile, staged columns, row pitch (floats)
    int GAP;           // extra input-row slots between two images of one tile
    int CC, Cpad, nchunks;
};

// fp32 tiled forward.  MODE: tconv_mode_t, CHAN: CH_SUM / CH_MAX / CH_MIN, WIN: emit winners.
// Q quads of 4 pixels per thread, KG groups of 8 output channels and PW pixel warps per CTA.
template <int MODE, int CHAN, bool WIN, int R, int S, int SW, int DW, int Q, int KG, int PW>
__global__ void __launch_bounds__(KG * PW * 32)
fwd_tiled_f32_kernel(const TiledParams p) {
    constexpr int RS = R * S;
    constexpr int TILE_K = KG * 8;
    constexpr int NT = KG * PW * 32;
    constexpr int L = 3 * SW + (S - 1) * DW + 1;  // input columns one quad touches per row
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool PAR = (MODE == TCONV_PARALLEL);
    constexpr bool TAP_MIN = (MODE == TCONV_MIN_PLUS);  // tap-level extremum of single-branch modes
    // running extremum carried across channels when tap and channel level agree
    constexpr bool CARRIED = !TWO && !WIN &&
                             ((MODE == TCONV_MAX_PLUS && CHAN == CH_MAX) ||
                              (MODE == TCONV_MIN_PLUS && CHAN == CH_MIN));
    const Geo& g = p.g;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int x_stage = p.CC * p.NSLOTS * p.XP;          // floats
    const int w_stage = p.CC * RS * TILE_K;              // floats
    const int ab_stage = TWO ? p.CC * TILE_K : 0;        // floats (each of alpha, beta)
    const int stage_floats = x_stage + w_stage * (PAR ? 2 : 1) + 2 * ab_stage;
    float* stage0 = reinterpret_cast<float*>(smem_raw);
    int* slot_off = reinterpret_cast<int*>(stage0 + 2 * stage_floats);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int kg = warp % KG, wp = warp / KG;
    const int ct = blockIdx.x % p.n_col_tiles;
    const int rt = blockIdx.x / p.n_col_tiles;
    const int kt = blockIdx.y;
    const int ow0 = ct * p.TW;
    const int row0 = rt * p.TH;
    const int iw0 = ow0 * SW - g.pw;
    const int n0 = row0 / g.OH;

    // input-row slot table: element offset of the row start inside x (per channel 0), or -1
    for (int sl = tid; sl < p.NSLOTS; sl += NT) slot_off[sl] = -1;
    __syncthreads();
    {
        const int rows_here = min(p.TH, p.total_rows - row0);
        const int span = (R - 1) * g.dh + 1;
        for (int e = tid; e < rows_here * span; e += NT) {
            const int lr = e / span, dr = e - lr * span;
            const int gr = row0 + lr;
            const int n = gr / g.OH, oh = gr - n * g.OH;
            const int ih = oh * g.sh - g.ph + dr;
            const int sl = lr * g.sh + (n - n0) * p.GAP + dr;
            if (ih >= 0 && ih < g.H) slot_off[sl] = (n * g.C * g.H + ih) * g.W;  // several writers, one value
        }
    }
    __syncthreads();

    // per-thread pixel quads
    int xoff[Q];
    int out_row[Q];   // flattened (n, oh) row, -1 if outside
    int qcol[Q];      // first output column of the quad
#pragma unroll
    for (int q = 0; q < Q; ++q) {
        const int qi = wp * 32 + lane + q * (32 * PW);
        int lr = qi / p.QPR;
        const int qx = qi - lr * p.QPR;
        const bool ok = (lr < p.TH) && (row0 + lr < p.total_rows);
        if (!ok) lr = 0;
        const int gr = row0 + lr;
        const int n = gr / g.OH;
        out_row[q] = ok ? gr : -1;
        qcol[q] = ow0 + qx * 4;
        xoff[q] = (lr * g.sh + (n - n0) * p.GAP) * p.XP + qx * 4 * SW;
    }

    const float* xg = reinterpret_cast<const float*>(p.x);
    const size_t chw = (size_t)g.H * g.W;
    const float* wt_k = p.wt + (size_t)kt * p.Cpad * RS * TILE_K;
    const float* wt2_k = PAR ? p.wt2 + (size_t)kt * p.Cpad * RS * TILE_K : nullptr;
    const float* at_k = TWO ? p.at + (size_t)kt * p.Cpad * TILE_K : nullptr;
    const float* bt_k = TWO ? p.bt + (size_t)kt * p.Cpad * TILE_K : nullptr;

    auto issue_chunk = [&](int ch, float* st) {
        const int c0 = ch * p.CC;
        // x halo tile: one warp per (channel, slot) row, lanes along the columns
        float* xs = st;
        for (int rowi = warp; rowi < p.CC * p.NSLOTS; rowi += KG * PW) {
            const int cc = rowi / p.NSLOTS, sl = rowi - cc * p.NSLOTS;
            const int off = slot_off[sl];
            const bool rok = (off >= 0) && (c0 + cc < g.C);
            const float* src_row = xg + (rok ? (size_t)off + (size_t)(c0 + cc) * chw : 0);
            float* dst_row = xs + (size_t)rowi * p.XP;
            for (int col = lane; col < p.XW; col += 32) {
                const int iw = iw0 + col;
                const bool ok = rok && iw >= 0 && iw < g.W;
                cp_async4(dst_row + col, ok ? src_row + iw : xg, ok);
            }
        }
        // weights (and alpha, beta): contiguous blocks, 16 bytes per copy
        float* ws = st + x_stage;
        const float* wsrc = wt_k + (size_t)c0 * RS * TILE_K;
        for (int e = tid; e < w_stage / 4; e += NT) cp_async16(ws + e * 4, wsrc + e * 4);
        if (PAR) {
            const float* wsrc2 = wt2_k + (size_t)c0 * RS * TILE_K;
            for (int e = tid; e < w_stage / 4; e += NT) cp_async16(ws + w_stage + e * 4, wsrc2 + e * 4);
        }
        if (TWO) {
            float* as = st + x_stage + w_stage * (PAR ? 2 : 1);
            for (int e = tid; e < ab_stage / 4; e += NT) {
                cp_async16(as + e * 4, at_k + (size_t)c0 * TILE_K + e * 4);
                cp_async16(as + ab_stage + e * 4, bt_k + (size_t)c0 * TILE_K + e * 4);
            }
        }
        cp_async_commit();
    };

    // accumulators
    float acc[8][Q][4];   // Sum forms: running sum; Max/Min combine: running best
    int cbest[WIN && CHAN != CH_SUM ? 8 : 1][Q][4];
#pragma unroll
    for (int k = 0; k < 8; ++k)
#pragma unroll
        for (int q = 0; q < Q; ++q)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[k][q][j] = (CHAN == CH_SUM) ? 0.0f : (CHAN == CH_MAX ? -INFINITY : INFINITY);
                if (WIN && CHAN != CH_SUM) cbest[k][q][j] = 0;
            }

    const size_t plane = (size_t)g.OH * g.OW;
    issue_chunk(0, stage0);
    for (int ch = 0; ch < p.nchunks; ++ch) {
        float* st = stage0 + (ch & 1) * stage_floats;
        if (ch + 1 < p.nchunks) {
            issue_chunk(ch + 1, stage0 + ((ch + 1) & 1) * stage_floats);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const float* xs = st;
        const float* ws = st + x_stage + kg * 8;
        const float* ws2 = ws + w_stage;
        const float* as = st + x_stage + w_stage * (PAR ? 2 : 1) + kg * 8;
        const int nc = min(p.CC, g.C - ch * p.CC);
        for (int cc = 0; cc < nc; ++cc) {
            // the R rows of input this thread's quads touch in channel cc
            float xr[Q][R][L];
#pragma unroll
            for (int q = 0; q < Q; ++q)
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float* src = xs + (size_t)cc * p.NSLOTS * p.XP + xoff[q] + r * g.dh * p.XP;
#pragma unroll
                    for (int i = 0; i + 4 <= L; i += 4) {
                        const float4 v = *reinterpret_cast<const float4*>(src + i);
                        xr[q][r][i] = v.x; xr[q][r][i + 1] = v.y; xr[q][r][i + 2] = v.z; xr[q][r][i + 3] = v.w;
                    }
                    if constexpr ((L & 3) >= 2) {
                        const float2 v = *reinterpret_cast<const float2*>(src + (L & ~3));
                        xr[q][r][L & ~3] = v.x; xr[q][r][(L & ~3) + 1] = v.y;
                    }
                    if constexpr (L & 1) xr[q][r][L - 1] = src[L - 1];
                }
            const float* wc = ws + (size_t)cc * RS * TILE_K;
            const float* wc2 = ws2 + (size_t)cc * RS * TILE_K;

            float mx[CARRIED ? 1 : 8][Q][4];           // per-channel extremum (max branch / single branch)
            float mn[TWO ? 8 : 1][Q][4];               // per-channel minimum (two-branch modes)
            int amx[WIN && CHAN == CH_SUM ? 8 : 1][Q][4], amn[WIN && TWO ? 8 : 1][Q][4];

            if constexpr (WIN && CHAN == CH_SUM) {
                // winner codes per (output, channel): every tap is compared on its own
#pragma unroll
                for (int tap = 0; tap < RS; ++tap) {
                    const int r = tap / S, s = tap % S;
                    float wv[8], wv2[8];
                    {
                        const float4 a = *reinterpret_cast<const float4*>(wc + tap * TILE_K);
                        const float4 b = *reinterpret_cast<const float4*>(wc + tap * TILE_K + 4);
                        wv[0] = a.x; wv[1] = a.y; wv[2] = a.z; wv[3] = a.w;
                        wv[4] = b.x; wv[5] = b.y; wv[6] = b.z; wv[7] = b.w;
                    }
                    if constexpr (PAR) {
                        const float4 a = *reinterpret_cast<const float4*>(wc2 + tap * TILE_K);
                        const float4 b = *reinterpret_cast<const float4*>(wc2 + tap * TILE_K + 4);
                        wv2[0] = a.x; wv2[1] = a.y; wv2[2] = a.z; wv2[3] = a.w;
                        wv2[4] = b.x; wv2[5] = b.y; wv2[6] = b.z; wv2[7] = b.w;
                    }
#pragma unroll
                    for (int q = 0; q < Q; ++q)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float xv = xr[q][r][j * SW + s * DW];
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const float t = __fadd_rn(xv, wv[k]);
                                const float t2 = PAR ? __fadd_rn(xv, wv2[k]) : t;
                                if constexpr (TWO) {
                                    if (tap == 0) {
                                        mn[k][q][j] = t; amn[k][q][j] = 0;
                                        mx[k][q][j] = t2; amx[k][q][j] = 0;
                                    } else {
                                        if (t < mn[k][q][j]) { mn[k][q][j] = t; amn[k][q][j] = tap; }
                                        if (t2 > mx[k][q][j]) { mx[k][q][j] = t2; amx[k][q][j] = tap; }
                                    }
                                } else {
                                    if (tap == 0) {
                                        mx[k][q][j] = t; amx[k][q][j] = 0;
                                    } else if (TAP_MIN ? (t < mx[k][q][j]) : (t > mx[k][q][j])) {
                                        mx[k][q][j] = t; amx[k][q][j] = tap;
                                    }
                                }
                            }
                        }
                }
            } else {
                // taps folded in groups: a fresh chain opens with 3 taps, later groups take 2
                constexpr int FIRST = CARRIED ? 2 : (RS >= 3 ? 3 : RS);
                constexpr int NG = 1 + (RS - FIRST + 1) / 2;
#pragma unroll
                for (int gi = 0; gi < NG; ++gi) {
                    const int t0 = (gi == 0) ? 0 : FIRST + 2 * (gi - 1);
                    const int nt = (gi == 0) ? (FIRST < RS ? FIRST : RS) : ((RS - t0) < 2 ? (RS - t0) : 2);
                    float wv[3][8], wv2[PAR ? 3 : 1][8];
#pragma unroll
                    for (int u = 0; u < 3; ++u)
                        if (u < nt) {
                            const float4 a = *reinterpret_cast<const float4*>(wc + (t0 + u) * TILE_K);
                            const float4 b = *reinterpret_cast<const float4*>(wc + (t0 + u) * TILE_K + 4);
                            wv[u][0] = a.x; wv[u][1] = a.y; wv[u][2] = a.z; wv[u][3] = a.w;
                            wv[u][4] = b.x; wv[u][5] = b.y; wv[u][6] = b.z; wv[u][7] = b.w;
                            if constexpr (PAR) {
                                const float4 c4 = *reinterpret_cast<const float4*>(wc2 + (t0 + u) * TILE_K);
                                const float4 d4 = *reinterpret_cast<const float4*>(wc2 + (t0 + u) * TILE_K + 4);
                                wv2[u][0] = c4.x; wv2[u][1] = c4.y; wv2[u][2] = c4.z; wv2[u][3] = c4.w;
                                wv2[u][4] = d4.x; wv2[u][5] = d4.y; wv2[u][6] = d4.z; wv2[u][7] = d4.w;
                            }
                        }
#pragma unroll
                    for (int q = 0; q < Q; ++q)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float xv[3];
#pragma unroll
                            for (int u = 0; u < 3; ++u)
                                if (u < nt) {
                                    const int tap = t0 + u;
                                    xv[u] = xr[q][tap / S][j * SW + (tap % S) * DW];
                                }
#pragma unroll
                            for (int kp = 0; kp < 4; ++kp) {
                                float ta[3][2], tb[3][2];
#pragma unroll
                                for (int u = 0; u < 3; ++u)
                                    if (u < nt) {
                                        add2(xv[u], wv[u][2 * kp], wv[u][2 * kp + 1], ta[u][0], ta[u][1]);
                                        if constexpr (PAR)
                                            add2(xv[u], wv2[u][2 * kp], wv2[u][2 * kp + 1], tb[u][0], tb[u][1]);
                                    }
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    const int k = 2 * kp + h;
                                    if constexpr (CARRIED) {
                                        float& m = acc[k][q][j];
                                        m = (nt == 2) ? ext3(m, ta[0][h], ta[1][h], TAP_MIN)
                                                      : ext2(m, ta[0][h], TAP_MIN);
                                    } else if constexpr (TWO) {
                                        float& lo = mn[k][q][j];
                                        float& hi = mx[k][q][j];
                                        const float (*tm)[2] = PAR ? tb : ta;
                                        if (gi == 0) {
                                            lo = nt == 3 ? ext3(ta[0][h], ta[1][h], ta[2][h], true)
                                                 : nt == 2 ? ext2(ta[0][h], ta[1][h], true) : ta[0][h];
                                            hi = nt == 3 ? ext3(tm[0][h], tm[1][h], tm[2][h], false)
                                                 : nt == 2 ? ext2(tm[0][h], tm[1][h], false) : tm[0][h];
                                        } else {
                                            lo = nt == 2 ? ext3(lo, ta[0][h], ta[1][h], true) : ext2(lo, ta[0][h], true);
                                            hi = nt == 2 ? ext3(hi, tm[0][h], tm[1][h], false) : ext2(hi, tm[0][h], false);
                                        }
                                    } else {
                                        float& m = mx[k][q][j];
                                        if (gi == 0)
                                            m = nt == 3 ? ext3(ta[0][h], ta[1][h], ta[2][h], TAP_MIN)
                                                : nt == 2 ? ext2(ta[0][h], ta[1][h], TAP_MIN) : ta[0][h];
                                        else
                                            m = nt == 2 ? ext3(m, ta[0][h], ta[1][h], TAP_MIN)
                                                        : ext2(m, ta[0][h], TAP_MIN);
                                    }
                                }
                            }
                        }
                }
            }

            // channel combine
            if constexpr (!CARRIED) {
                float av[8], bv[8];
                if constexpr (TWO) {
                    const float4 a0 = *reinterpret_cast<const float4*>(as + cc * TILE_K);
                    const float4 a1 = *reinterpret_cast<const float4*>(as + cc * TILE_K + 4);
                    const float4 b0 = *reinterpret_cast<const float4*>(as + ab_stage + cc * TILE_K);
                    const float4 b1 = *reinterpret_cast<const float4*>(as + ab_stage + cc * TILE_K + 4);
                    av[0] = a0.x; av[1] = a0.y; av[2] = a0.z; av[3] = a0.w;
                    av[4] = a1.x; av[5] = a1.y; av[6] = a1.z; av[7] = a1.w;
                    bv[0] = b0.x; bv[1] = b0.y; bv[2] = b0.z; bv[3] = b0.w;
                    bv[4] = b1.x; bv[5] = b1.y; bv[6] = b1.z; bv[7] = b1.w;
                }
                const int c = ch * p.CC + cc;
#pragma unroll
                for (int k = 0; k < 8; ++k)
#pragma unroll
                    for (int q = 0; q < Q; ++q)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if constexpr (TWO) {
                                acc[k][q][j] = __fmaf_rn(av[k], mn[k][q][j], acc[k][q][j]);
                                acc[k][q][j] = __fmaf_rn(bv[k], mx[k][q][j], acc[k][q][j]);
                            } else if constexpr (CHAN == CH_SUM) {
                                acc[k][q][j] = __fadd_rn(acc[k][q][j], mx[k][q][j]);
                            } else if constexpr (WIN) {
                                const bool better = (CHAN == CH_MAX) ? (mx[k][q][j] > acc[k][q][j])
                                                                     : (mx[k][q][j] < acc[k][q][j]);
                                if (better) { acc[k][q][j] = mx[k][q][j]; cbest[k][q][j] = c; }
                            } else {
                                acc[k][q][j] = ext2(acc[k][q][j], mx[k][q][j], CHAN == CH_MIN);
                            }
                        }
                if constexpr (WIN && CHAN == CH_SUM) {
                    // one byte per (n, k, c, oh, ow): low nibble argmin tap, high nibble argmax tap
                    uint8_t* codes = reinterpret_cast<uint8_t*>(p.winners);
#pragma unroll
                    for (int q = 0; q < Q; ++q) {
                        if (out_row[q] < 0) continue;
                        const int n = out_row[q] / g.OH, oh = out_row[q] - n * g.OH;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const int kk = kt * TILE_K + kg * 8 + k;
                            if (kk >= g.K) continue;
                            uint8_t* dst = codes + (((size_t)n * g.K + kk) * g.C + c) * plane +
                                           (size_t)oh * g.OW + qcol[q];
                            unsigned packed = 0;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                unsigned code;
                                if constexpr (TWO) code = amn[k][q][j] | (amx[k][q][j] << 4);
                                else code = TAP_MIN ? amx[k][q][j] : (amx[k][q][j] << 4);
                                packed |= code << (8 * j);
                            }
                            if (qcol[q] + 3 < g.OW && ((g.OW & 3) == 0)) {
                                *reinterpret_cast<unsigned*>(dst) = packed;
                            } else {
#pragma unroll
                                for (int j = 0; j < 4; ++j)
                                    if (qcol[q] + j < g.OW) dst[j] = (uint8_t)(packed >> (8 * j));
                            }
                        }
                    }
                }
            }
        }
        __syncthreads();
    }

    // epilogue: bias, store, winner index of the Max / Min channel combines
    float* yg = reinterpret_cast<float*>(p.y);
#pragma unroll
    for (int q = 0; q < Q; ++q) {
        if (out_row[q] < 0) continue;
        const int n = out_row[q] / g.OH, oh = out_row[q] - n * g.OH;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int kk = kt * TILE_K + kg * 8 + k;
            if (kk >= g.K) continue;
            const float bk = p.bias ? p.bias[kk] : 0.0f;
            const size_t o = ((size_t)n * g.K + kk) * plane + (size_t)oh * g.OW + qcol[q];
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = p.bias ? __fadd_rn(acc[k][q][j], bk) : acc[k][q][j];
            if (yg) {
                if (qcol[q] + 3 < g.OW && ((g.OW & 3) == 0)) {
                    *reinterpret_cast<float4*>(yg + o) = make_float4(v[0], v[1], v[2], v[3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (qcol[q] + j < g.OW) yg[o + j] = v[j];
                }
            }
            if constexpr (WIN && CHAN != CH_SUM) {
                // the winning channel is known; rescan its window for the first tap that attains the
                // extremum (same adds as the main loop, so equality is exact)
                int32_t* idx = reinterpret_cast<int32_t*>(p.winners);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int ow = qcol[q] + j;
                    if (ow >= g.OW) continue;
                    const int c = cbest[k][q][j];
                    const float* xc = xg + ((size_t)n * g.C + c) * chw;
                    const float* wk = wt_k + ((size_t)c * RS) * TILE_K + kg * 8 + k;
                    int tapw = 0;
#pragma unroll
                    for (int tap = RS - 1; tap >= 0; --tap) {
                        const int ih = oh * g.sh - g.ph + (tap / S) * g.dh;
                        const int iw = ow * SW - g.pw + (tap % S) * DW;
                        const float xv = (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) ? xc[(size_t)ih * g.W + iw] : 0.0f;
                        if (__fadd_rn(xv, wk[tap * TILE_K]) == acc[k][q][j]) tapw = tap;
                    }
                    idx[o + j] = c * RS + tapw;
                }
            }
        }
    }
}

// ----------------------------------------------------------------------------------
// host side: tile selection and launch
struct TiledPlan {
    TiledParams p;
    dim3 grid;
    int threads;
    size_t smem;
    int tile_k;
    size_t ws_w, ws_ab;  // workspace split (bytes): each weight array, each of alpha / beta
};

inline size_t tiled_ws_bytes(const Geo& g) {
    // upper bound over every tile choice: K padded to 64, C padded to 8
    const size_t Kp = ((size_t)g.K + 63) / 64 * 64, Cp = ((size_t)g.C + 7) / 8 * 8;
    const size_t w = Kp * Cp * g.RS * sizeof(float);
    const size_t ab = Kp * Cp * sizeof(float);
    return 2 * w + 2 * ab + 1024;
}

template <int R, int S, int SW, int DW, int Q, int KG, int PW>
inline bool plan_tiles(const Geo& g, bool par, bool two, TiledPlan* pl) {
    TiledParams& p = pl->p;
    constexpr int TILE_K = KG * 8;
    constexpr int NQ = Q * 32 * PW;
    const int qpr_full = (g.OW + 3) / 4;
    // column tiles: as wide as the row allows, at most NQ/2 quads (so a tile keeps >= 2 rows
    // unless the row is very wide), split evenly
    int max_qpr = NQ >= 32 ? NQ / 4 : NQ;
    if (max_qpr < 1) max_qpr = 1;
    const int ncol = (qpr_full + max_qpr - 1) / max_qpr;
    p.QPR = (qpr_full + ncol - 1) / ncol;
    p.TW = p.QPR * 4;
    p.n_col_tiles = (g.OW + p.TW - 1) / p.TW;
    p.TH = NQ / p.QPR;
    if (p.TH < 1) return false;
    p.total_rows = g.N * g.OH;
    if (p.TH > p.total_rows) p.TH = p.total_rows;
    p.n_row_tiles = (p.total_rows + p.TH - 1) / p.TH;
    p.GAP = (R - 1) * g.dh - g.sh + 1;
    if (p.GAP < 0) p.GAP = 0;
    const int max_imgs = (p.TH - 1) / g.OH + 2;
    p.NSLOTS = (p.TH - 1) * g.sh + (R - 1) * g.dh + 1 + (max_imgs - 1) * p.GAP;
    p.XW = (p.TW - 1) * SW + (S - 1) * DW + 1;
    // a quad reads up to 3*SW + (S-1)*DW + 1 floats from column 4*SW*qx, rounded up to vectors
    const int reach = (p.QPR - 1) * 4 * SW + ((3 * SW + (S - 1) * DW + 1 + 3) & ~3);
    p.XP = ((reach > p.XW ? reach : p.XW) + 3) & ~3;
    p.CC = 8;
    p.Cpad = (g.C + p.CC - 1) / p.CC * p.CC;
    p.nchunks = p.Cpad / p.CC;
    const size_t stage = (size_t)p.CC * p.NSLOTS * p.XP + (size_t)p.CC * g.RS * TILE_K * (par ? 2 : 1) +
                         (two ? 2 * (size_t)p.CC * TILE_K : 0);
    pl->smem = 2 * stage * sizeof(float) + (size_t)p.NSLOTS * sizeof(int) + 16;
    if (pl->smem > 200 * 1024) return false;
    const int nkt = (g.K + TILE_K - 1) / TILE_K;
    pl->grid = dim3((unsigned)(p.n_col_tiles * p.n_row_tiles), (unsigned)nkt, 1);
    pl->threads = KG * PW * 32;
    pl->tile_k = TILE_K;
    pl->ws_w = (size_t)nkt * p.Cpad * g.RS * TILE_K * sizeof(float);
    pl->ws_ab = (size_t)nkt * p.Cpad * TILE_K * sizeof(float);
    return true;
}

template <typename T, int MODE, int CHAN, bool WIN, int R, int S, int SW, int DW, int Q, int KG, int PW>
int launch_tiled_variant(const Geo& g, const T* x, const T* w, const T* w2, const float* alpha,
                         const float* beta, const float* bias, T* y, void* winners, void* ws,
                         size_t ws_bytes, cudaStream_t st) {
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool PAR = (MODE == TCONV_PARALLEL);
    TiledPlan pl;
    pl.p.g = g;
    if (!plan_tiles<R, S, SW, DW, Q, KG, PW>(g, PAR, TWO, &pl)) return TCONV_ERR_UNSUPPORTED;
    const size_t need = pl.ws_w * (PAR ? 2 : 1) + (TWO ? 2 * pl.ws_ab : 0);
    if (!ws || ws_bytes < need) return TCONV_ERR_WORKSPACE_TOO_SMALL;
    float* wt = reinterpret_cast<float*>(ws);
    float* wt2 = PAR ? wt + pl.ws_w / sizeof(float) : nullptr;
    float* at = TWO ? wt + (pl.ws_w * (PAR ? 2 : 1)) / sizeof(float) : nullptr;
    float* bt = TWO ? at + pl.ws_ab / sizeof(float) : nullptr;
    const int nkt = pl.grid.y;
    const size_t nrep = (size_t)nkt * pl.p.Cpad * g.RS * pl.tile_k;
    repack_weights_kernel<T><<<(unsigned)((nrep + 255) / 256), 256, 0, st>>>(
        g.K, g.C, g.RS, pl.tile_k, pl.p.Cpad, nkt, w, w2, alpha, beta, wt, wt2, at, bt);
    pl.p.x = x; pl.p.wt = wt; pl.p.wt2 = wt2; pl.p.at = at; pl.p.bt = bt;
    pl.p.bias = bias; pl.p.y = y; pl.p.winners = winners;
    auto kern = fwd_tiled_f32_kernel<MODE, CHAN, WIN, R, S, SW, DW, Q, KG, PW>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
        return TCONV_ERR_CUDA;
    kern<<<pl.grid, pl.threads, pl.smem, st>>>(pl.p);
    return TCONV_OK;
}

// Geometry families with a tiled kernel: 3x3 windows with (stride_w, dil_w) in
// {(1,1), (2,1), (1,2)}.
template <typename T, int MODE, int CHAN, bool WIN>
int launch_tiled_geom(const Geo& g, const T* x, const T* w, const T* w2, const float* alpha,
                      const float* beta, const float* bias, T* y, void* winners, void* ws,
                      size_t ws_bytes, cudaStream_t st) {
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    // two quads per thread where one running value per output suffices (the carried
    // extremum of layers (iv), (v) without winners), else one
    constexpr bool CARRIED = !TWO && !WIN && ((MODE == TCONV_MAX_PLUS && CHAN == CH_MAX) ||
                                              (MODE == TCONV_MIN_PLUS && CHAN == CH_MIN));
    constexpr int Q = CARRIED ? 2 : 1;
    if (g.R == 3 && g.S == 3) {
        if (g.sw == 1 && g.dw == 1)
            return launch_tiled_variant<T, MODE, CHAN, WIN, 3, 3, 1, 1, Q, 4, 1>(g, x, w, w2, alpha, beta, bias, y, winners, ws, ws_bytes, st);
        if (g.sw == 2 && g.dw == 1)
            return launch_tiled_variant<T, MODE, CHAN, WIN, 3, 3, 2, 1, Q, 4, 1>(g, x, w, w2, alpha, beta, bias, y, winners, ws, ws_bytes, st);
        if (g.sw == 1 && g.dw == 2)
            return launch_tiled_variant<T, MODE, CHAN, WIN, 3, 3, 1, 2, Q, 4, 1>(g, x, w, w2, alpha, beta, bias, y, winners, ws, ws_bytes, st);
    }
    return TCONV_ERR_UNSUPPORTED;
}

template <typename T, bool WIN>
int launch_tiled_mode(const Geo& g, const T* x, const T* w, const T* w2, const float* alpha,
                      const float* beta, const float* bias, T* y, void* winners, void* ws,
                      size_t ws_bytes, cudaStream_t st) {
#define TCONV_GO(M, CH) \
    return launch_tiled_geom<T, M, CH, WIN>(g, x, w, w2, alpha, beta, bias, y, winners, ws, ws_bytes, st)
    if (g.mode == TCONV_COMPOUND) TCONV_GO(TCONV_COMPOUND, CH_SUM);
    if (g.mode == TCONV_PARALLEL) TCONV_GO(TCONV_PARALLEL, CH_SUM);
    if (g.mode == TCONV_MAX_PLUS) {
        if (g.chan == CH_MAX) TCONV_GO(TCONV_MAX_PLUS, CH_MAX);
        if (g.chan == CH_MIN) TCONV_GO(TCONV_MAX_PLUS, CH_MIN);
        TCONV_GO(TCONV_MAX_PLUS, CH_SUM);
    }
    if (g.chan == CH_MAX) TCONV_GO(TCONV_MIN_PLUS, CH_MAX);
    if (g.chan == CH_MIN) TCONV_GO(TCONV_MIN_PLUS, CH_MIN);
    TCONV_GO(TCONV_MIN_PLUS, CH_SUM);
#undef TCONV_GO
}

// Launches the tiled forward kernel that covers this geometry.  Returns
// TCONV_ERR_UNSUPPORTED when none does (the caller then uses the any-shape kernel).
template <typename T>
int launch_fwd_tiled(const Geo& g, const T* x, const T* w, const T* w2, const float* alpha,
                     const float* beta, const float* bias, T* y, void* winners, void* ws,
                     size_t ws_bytes, cudaStream_t st, const char** name) {
    if constexpr (sizeof(T) != 4) {
        return TCONV_ERR_UNSUPPORTED;  // bf16: separate kernel
    } else {
    if (g.wide) return TCONV_ERR_UNSUPPORTED;
    if ((double)g.N * g.C * g.H * g.W >= 2.0e9) return TCONV_ERR_UNSUPPORTED;  // 32-bit offsets
    *name = winners ? "fwd_tiled_f32_win" : "fwd_tiled_f32";
    if (winners)
        return launch_tiled_mode<T, true>(g, x, w, w2, alpha, beta, bias, y, winners, ws, ws_bytes, st);
    return launch_tiled_mode<T, false>(g, x, w, w2, alpha, beta, bias, y, winners, ws, ws_bytes, st);
    }
}

}  // namespace tconv

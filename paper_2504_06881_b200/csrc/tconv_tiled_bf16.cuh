// Tiled forward kernels (bf16): same tiling and staging as the fp32 kernels, with the
// arithmetic on packed pairs.  A 32-bit register holds two horizontally adjacent output
// pixels of one output channel; the weights are repacked as {w, w} pairs, so one
// add.bf16x2 forms two tap sums and one min/max.bf16x2 folds them.  Every tap sum is a
// single rounded bf16 add, min / max are exact, and the channel combine runs in fp32
// (packed fp32 fused multiply-adds over the pixel pair).
#pragma once
#include "tconv_tiled.cuh"

namespace tconv {

__device__ __forceinline__ unsigned hadd2u(unsigned a, unsigned b) {
    unsigned d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ unsigned hext2u(unsigned a, unsigned b, bool is_min) {
    unsigned d;
    if (is_min) asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    else asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ __nv_bfloat162 as_bf162(unsigned u) {
    return *reinterpret_cast<__nv_bfloat162*>(&u);
}
// per half: 0xFFFF where a > b (a < b when is_min)
__device__ __forceinline__ unsigned hbetter_mask(unsigned a, unsigned b, bool is_min) {
    return is_min ? __hlt2_mask(as_bf162(a), as_bf162(b)) : __hgt2_mask(as_bf162(a), as_bf162(b));
}
__device__ __forceinline__ float bf_lo(unsigned u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(unsigned u) { return __uint_as_float(u & 0xffff0000u); }
// {c0, c1} = a * {v0, v1} + {c0, c1}, each lane one fused multiply-add
__device__ __forceinline__ void fma2(float a, float v0, float v1, float& c0, float& c1) {
    unsigned long long aa, vv, cc;
    asm("mov.b64 %0, {%1, %1};" : "=l"(aa) : "f"(a));
    asm("mov.b64 %0, {%1, %2};" : "=l"(vv) : "f"(v0), "f"(v1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(cc) : "f"(c0), "f"(c1));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(cc) : "l"(aa), "l"(vv));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(c0), "=f"(c1) : "l"(cc));
}
__device__ __forceinline__ void addpair(float v0, float v1, float& c0, float& c1) {
    unsigned long long vv, cc;
    asm("mov.b64 %0, {%1, %2};" : "=l"(vv) : "f"(v0), "f"(v1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(cc) : "f"(c0), "f"(c1));
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(cc) : "l"(vv));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(c0), "=f"(c1) : "l"(cc));
}

// NW 32-bit words starting at word START past a pointer aligned to ALIGN words.
template <int ALIGN, int START, int NW, int I = 0>
__device__ __forceinline__ void load_words(const unsigned* base, unsigned* out) {
    if constexpr (I < NW) {
        constexpr int pos = START + I;
        if constexpr ((ALIGN % 4 == 0) && (pos % 4 == 0) && (I + 4 <= NW)) {
            const uint4 v = *reinterpret_cast<const uint4*>(base + pos);
            out[I] = v.x; out[I + 1] = v.y; out[I + 2] = v.z; out[I + 3] = v.w;
            load_words<ALIGN, START, NW, I + 4>(base, out);
        } else if constexpr ((pos % 2 == 0) && (I + 2 <= NW)) {
            const uint2 v = *reinterpret_cast<const uint2*>(base + pos);
            out[I] = v.x; out[I + 1] = v.y;
            load_words<ALIGN, START, NW, I + 2>(base, out);
        } else {
            out[I] = base[pos];
            load_words<ALIGN, START, NW, I + 1>(base, out);
        }
    }
}
// The pixel pair whose first element sits E elements past the first loaded word:
// elements (E, E + SW).
template <int SW, int E>
__device__ __forceinline__ unsigned pixel_pair(const unsigned* xw) {
    if constexpr (SW == 1) {
        if constexpr (E % 2 == 0) return xw[E / 2];
        else return __byte_perm(xw[E / 2], xw[E / 2 + 1], 0x5432);
    } else {
        return __byte_perm(xw[E / 2], xw[E / 2 + 1], (E % 2) ? 0x7632 : 0x5410);
    }
}

// Weight repack for the bf16 kernels: every weight becomes the pair {w, w}.  (A template so
// that each translation unit that includes this header gets its own instance.)
template <int UNUSED = 0>
__global__ void repack_weights_bf16_kernel(int K, int C, int RS, int tile_k, int Cpad, int nkt,
                                           const __nv_bfloat16* __restrict__ w,
                                           const __nv_bfloat16* __restrict__ w2,
                                           const float* __restrict__ alpha,
                                           const float* __restrict__ beta, unsigned* __restrict__ wt,
                                           unsigned* __restrict__ wt2, float* __restrict__ at,
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
        const unsigned short* w16 = reinterpret_cast<const unsigned short*>(w);
        const unsigned a = ok ? w16[src] : 0u;
        wt[i] = a | (a << 16);
        if (wt2) {
            const unsigned b = ok ? reinterpret_cast<const unsigned short*>(w2)[src] : 0u;
            wt2[i] = b | (b << 16);
        }
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

// Element i of x as bf16 bits: x holds bf16, or float values that are rounded to nearest even here
// (the same rounding a conversion of the whole tensor would apply).
__device__ __forceinline__ unsigned short load_x(const unsigned short* x, size_t i, int xf32) {
    if (!xf32) return x[i];
    return __bfloat16_as_ushort(__float2bfloat16_rn(reinterpret_cast<const float*>(x)[i]));
}

// KPT words of packed weights of one tap (one or two 16-byte loads)
template <int KPT>
__device__ __forceinline__ void loadw(const unsigned* p, unsigned* out) {
    const uint4 a = *reinterpret_cast<const uint4*>(p);
    out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
    if constexpr (KPT == 8) {
        const uint4 b = *reinterpret_cast<const uint4*>(p + 4);
        out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
    }
}

// KPT: output channels per thread, 8, or 4 for layers that would otherwise keep too few warps
// resident (small maps with many channels at a small batch).
template <int MODE, int CHAN, bool WIN, bool XTMA, bool RAG, int R, int S, int SW, int DW, int Q, int KG, int PW, int KPT = 8,
          bool STATS = false>
__global__ void __launch_bounds__(KG * PW * 32)
fwd_tiled_bf16_kernel(const __grid_constant__ CUtensorMap xmap, const TiledParams p) {
    static_assert(S == 3, "the pixel-pair selection below is written for 3 taps per row");
    static_assert(KPT == 8 || KPT == 4, "output channels per thread");
    constexpr int RS = R * S;
    constexpr int TILE_K = KG * KPT;
    constexpr int NT = KG * PW * 32;
    constexpr int NWARPS = KG * PW;
    constexpr int L = 3 * SW + (S - 1) * DW + 1;   // input elements one quad touches per row
    constexpr int SHIFT = XTMA ? TmaShift<S, DW, 2>::value : 0;
    constexpr int WSTART = SHIFT / 2;               // first word of the segment
    constexpr int NW = (SHIFT + L - 1) / 2 - SHIFT / 2 + 1;
    constexpr int EODD = SHIFT & 1;                 // offset of the segment inside its first word
    constexpr int ALIGNW = (SW % 2 == 0) ? 4 : 2;   // word alignment of a quad's row pointer
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool PAR = (MODE == TCONV_PARALLEL);
    constexpr bool TAP_MIN = (MODE == TCONV_MIN_PLUS);
    constexpr bool CARRIED = !TWO && !WIN &&
                             ((MODE == TCONV_MAX_PLUS && CHAN == CH_MAX) ||
                              (MODE == TCONV_MIN_PLUS && CHAN == CH_MIN));
    constexpr bool SUMF = (CHAN == CH_SUM);
    const Geo& g = p.g;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned* stage0 = reinterpret_cast<unsigned*>(smem_raw);
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(stage0 + 2 * p.stage_floats);
    int* slot_off = reinterpret_cast<int*>(bars + 2);
    int* src_tab = slot_off + ((p.NSLOTS + 3) & ~3);   // staging table of the non-TMA path

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int kg = warp % KG, wp = warp / KG;
    const int ct = blockIdx.x % p.n_col_tiles;
    const int rt = blockIdx.x / p.n_col_tiles;
    const int kt = blockIdx.y;
    const int ow0 = ct * p.TW;
    constexpr int NQ_TILE = Q * 32 * PW;   // quads per tile
    int row0, rows_here, qfirst = 0;       // qfirst: ragged tiles start this many quads into row0
    if constexpr (RAG) {
        const int q0 = rt * NQ_TILE;
        row0 = q0 / p.QPR;
        qfirst = q0 - row0 * p.QPR;
        rows_here = (min(q0 + NQ_TILE, p.total_quads) - 1) / p.QPR - row0 + 1;
    } else if (p.tiles_per_img > 0) {
        const int n = rt / p.tiles_per_img;
        const int oh0 = (rt - n * p.tiles_per_img) * p.TH;
        row0 = n * g.OH + oh0;
        rows_here = min(p.TH, g.OH - oh0);
    } else {
        row0 = rt * p.TH;
        rows_here = min(p.TH, p.total_rows - row0);
    }
    const int iw0 = ow0 * SW - g.pw;
    const int n0 = row0 / g.OH;
    const int oh_first = row0 - n0 * g.OH;
    // a ragged TMA tile may run into the next image, which is staged as a second block
    const bool two_imgs = XTMA && RAG && (row0 + rows_here - 1) / g.OH > n0;

    if constexpr (XTMA) {
        if (tid == 0) {
            mbar_init(&bars[0], 1);
            mbar_init(&bars[1], 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
    } else {
        for (int sl = tid; sl < p.NSLOTS; sl += NT) slot_off[sl] = -1;
        __syncthreads();
        const int span = (R - 1) * g.dh + 1;
        for (int e = tid; e < rows_here * span; e += NT) {
            const int lr = e / span, dr = e - lr * span;
            const int gr = row0 + lr;
            const int n = gr / g.OH, oh = gr - n * g.OH;
            const int ih = oh * g.sh - g.ph + dr;
            const int sl = lr * g.sh + (n - n0) * p.GAP + dr;
            if (ih >= 0 && ih < g.H) slot_off[sl] = (n * g.C * g.H + ih) * g.W;
        }
        __syncthreads();
        // element offsets inside x (channel 0 of the tile's first image row space), -1 = zero
        for (int i = tid; i < p.NSLOTS * p.XP; i += NT) {
            const int sl = i / p.XP, col = i - sl * p.XP;
            const int iw = iw0 + col;
            const int off = slot_off[sl];
            src_tab[i] = (off >= 0 && iw >= 0 && iw < g.W) ? off + iw : -1;
        }
    }
    __syncthreads();

    int xoff[Q];      // word offset of the quad's row pointer inside a channel plane of the tile
    int out_row[Q];
    int qcol[Q];
    const int pitch_w = p.XP / 2;   // words per staged row
#pragma unroll
    for (int q = 0; q < Q; ++q) {
        const int qi = wp * 32 + lane + q * (32 * PW);
        const int qq = qi + qfirst;
        int lr = qq / p.QPR;
        const int qx = qq - lr * p.QPR;
        const bool ok = RAG ? (rt * NQ_TILE + qi < p.total_quads) : (lr < rows_here);
        if (!ok) lr = 0;
        const int gr = row0 + lr;
        const int n = gr / g.OH;
        out_row[q] = ok ? gr : -1;
        qcol[q] = ow0 + qx * 4;
        if constexpr (XTMA && RAG)
            xoff[q] = (n == n0 ? lr * g.sh * pitch_w : p.xblock / 2 + (gr - (n0 + 1) * g.OH) * g.sh * pitch_w) + qx * 2 * SW;
        else
            xoff[q] = (lr * g.sh + (n - n0) * p.GAP) * pitch_w + qx * 2 * SW;
    }

    const unsigned short* xg = reinterpret_cast<const unsigned short*>(p.x);
    const size_t chw = (size_t)g.H * g.W;
    const unsigned* wt_k = reinterpret_cast<const unsigned*>(p.wt) + (size_t)kt * p.Cpad * RS * TILE_K;
    const unsigned* wt2_k = PAR ? reinterpret_cast<const unsigned*>(p.wt2) + (size_t)kt * p.Cpad * RS * TILE_K : nullptr;
    const float* at_k = TWO ? p.at + (size_t)kt * p.Cpad * TILE_K : nullptr;
    const float* bt_k = TWO ? p.bt + (size_t)kt * p.Cpad * TILE_K : nullptr;
    const int w_off = p.x_stage, w2_off = p.x_stage + p.w_stage;
    const int a_off = p.x_stage + p.w_stage * (PAR ? 2 : 1), b_off = a_off + p.ab_stage;

    auto issue_chunk = [&](int ch, int s) {
        unsigned* st = stage0 + s * p.stage_floats;
        const int c0 = ch * p.CC;
        if constexpr (XTMA) {
            if (tid == 0 && !(p.debug_drop && ch == 0)) {
                const unsigned bytes = (unsigned)(p.xbox * 2 * (two_imgs ? 2 : 1) +
                                                  (p.w_stage * (PAR ? 2 : 1) + 2 * p.ab_stage) * 4);
                mbar_expect_tx(&bars[s], bytes);
                tma_load_3d(st, &xmap, iw0 - SHIFT, oh_first * g.sh - g.ph, n0 * g.C + c0, &bars[s]);
                if (two_imgs) tma_load_3d(st + p.xblock / 2, &xmap, iw0 - SHIFT, -g.ph, (n0 + 1) * g.C + c0, &bars[s]);
                bulk_load(st + w_off, wt_k + (size_t)c0 * RS * TILE_K, p.w_stage * 4, &bars[s]);
                if (PAR) bulk_load(st + w2_off, wt2_k + (size_t)c0 * RS * TILE_K, p.w_stage * 4, &bars[s]);
                if (TWO) {
                    bulk_load(st + a_off, at_k + (size_t)c0 * TILE_K, p.ab_stage * 4, &bars[s]);
                    bulk_load(st + b_off, bt_k + (size_t)c0 * TILE_K, p.ab_stage * 4, &bars[s]);
                }
            }
        } else {
            // x halo tile by plain 2-byte loads (rows are not 16-byte multiples here): the source
            // offset of every element of one channel plane comes from a table built once per CTA,
            // and the loads of the chunk's channels are issued together before any is stored
            unsigned short* xs = reinterpret_cast<unsigned short*>(st);
            const int per_c = p.NSLOTS * p.XP;
            const unsigned short pad_bits = (unsigned short)(g.neutral ? 0x7fc0 : 0);   // padding: zero, or NaN (skipped by min / max)
            for (int i = tid; i < per_c; i += NT) {
                const int so = src_tab[i];
                unsigned short v[8];
#pragma unroll
                for (int cc = 0; cc < 8; ++cc)
                    v[cc] = (cc < p.CC && c0 + cc < g.C) ? (so >= 0 ? load_x(xg, (size_t)(c0 + cc) * chw + so, g.xf32) : pad_bits)
                                                          : (unsigned short)0;
#pragma unroll
                for (int cc = 0; cc < 8; ++cc)
                    if (cc < p.CC) xs[cc * per_c + i] = v[cc];
            }
            const unsigned* wsrc = wt_k + (size_t)c0 * RS * TILE_K;
            for (int e = tid; e < p.w_stage / 4; e += NT) cp_async16(st + w_off + e * 4, wsrc + e * 4);
            if (PAR) {
                const unsigned* wsrc2 = wt2_k + (size_t)c0 * RS * TILE_K;
                for (int e = tid; e < p.w_stage / 4; e += NT) cp_async16(st + w2_off + e * 4, wsrc2 + e * 4);
            }
            if (TWO) {
                for (int e = tid; e < p.ab_stage / 4; e += NT) {
                    cp_async16(st + a_off + e * 4, at_k + (size_t)c0 * TILE_K + e * 4);
                    cp_async16(st + b_off + e * 4, bt_k + (size_t)c0 * TILE_K + e * 4);
                }
            }
            cp_async_commit();
        }
    };

    // running state: fp32 sums (Sum forms) or packed running best (Max / Min combine)
    float acc[SUMF ? KPT : 1][Q][4];
    unsigned best[SUMF ? 1 : KPT][Q][2];
    unsigned cbest[(WIN && !SUMF) ? KPT : 1][Q][2];   // winning channel per pixel, two 16-bit fields
    constexpr unsigned kNegInf2 = 0xFF80FF80u, kPosInf2 = 0x7F807F80u;
#pragma unroll
    for (int k = 0; k < KPT; ++k)
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            if constexpr (SUMF) {
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[k][q][j] = 0.0f;
            } else {
                best[k][q][0] = best[k][q][1] = (CHAN == CH_MAX) ? kNegInf2 : kPosInf2;
                if constexpr (WIN) cbest[k][q][0] = cbest[k][q][1] = 0u;
            }
        }

    const size_t plane = (size_t)g.OH * g.OW;
    const int row_step = g.dh * pitch_w;
    const int chan_step = p.NSLOTS * pitch_w;
    issue_chunk(0, 0);
    for (int ch = 0; ch < p.nchunks; ++ch) {
        const int s = ch & 1;
        unsigned* st = stage0 + s * p.stage_floats;
        if (ch + 1 < p.nchunks) issue_chunk(ch + 1, s ^ 1);
        if constexpr (XTMA) {
            if (!mbar_wait(&bars[s], (ch >> 1) & 1)) {
                if (p.status) *p.status = 1;
                mbar_wait(&bars[s], (ch >> 1) & 1);
                if (ch + 1 < p.nchunks) mbar_wait(&bars[s ^ 1], ((ch + 1) >> 1) & 1);
                return;
            }
        } else {
            if (ch + 1 < p.nchunks) cp_async_wait<1>(); else cp_async_wait<0>();
            __syncthreads();
        }
        const unsigned* ws = st + w_off + kg * KPT;
        const unsigned* ws2 = st + w2_off + kg * KPT;
        const float* as = reinterpret_cast<const float*>(st + a_off) + kg * KPT;
        const float* bs = reinterpret_cast<const float*>(st + b_off) + kg * KPT;
        const int nc = min(p.CC, g.C - ch * p.CC);
        for (int cc = 0; cc < nc; ++cc) {
            unsigned xw[Q][R][NW];
#pragma unroll
            for (int q = 0; q < Q; ++q)
#pragma unroll
                for (int r = 0; r < R; ++r)
                    load_words<ALIGNW, WSTART, NW>(st + cc * chan_step + xoff[q] + r * row_step, xw[q][r]);
            const unsigned* wc = ws + cc * (RS * TILE_K);
            const unsigned* wc2 = ws2 + cc * (RS * TILE_K);
            const int c = ch * p.CC + cc;

            unsigned mx[CARRIED ? 1 : KPT][Q][2];
            unsigned mn[TWO ? KPT : 1][Q][2];
            unsigned amx[(WIN && SUMF) ? KPT : 1][Q][2], amn[(WIN && TWO) ? KPT : 1][Q][2];

            if constexpr (WIN && SUMF) {
#pragma unroll
                for (int tap = 0; tap < RS; ++tap) {
                    constexpr unsigned one2 = 0x00010001u;
                    const unsigned tap2 = one2 * (unsigned)tap;
                    const int r = tap / S, sx = tap % S;
                    unsigned wv[KPT], wv2[KPT];
                    loadw<KPT>(wc + tap * TILE_K, wv);
                    if constexpr (PAR) loadw<KPT>(wc2 + tap * TILE_K, wv2);
#pragma unroll
                    for (int q = 0; q < Q; ++q)
#pragma unroll
                        for (int pp = 0; pp < 2; ++pp) {
                            unsigned xp;
                            // compile-time element offset of this pair: unrolled over (sx, pp)
                            if (sx == 0) xp = pp == 0 ? pixel_pair<SW, EODD + 0 * SW + 0 * DW>(xw[q][r]) : pixel_pair<SW, EODD + 2 * SW + 0 * DW>(xw[q][r]);
                            else if (sx == 1) xp = pp == 0 ? pixel_pair<SW, EODD + 0 * SW + 1 * DW>(xw[q][r]) : pixel_pair<SW, EODD + 2 * SW + 1 * DW>(xw[q][r]);
                            else xp = pp == 0 ? pixel_pair<SW, EODD + 0 * SW + 2 * DW>(xw[q][r]) : pixel_pair<SW, EODD + 2 * SW + 2 * DW>(xw[q][r]);
#pragma unroll
                            for (int k = 0; k < KPT; ++k) {
                                const unsigned t = hadd2u(xp, wv[k]);
                                const unsigned t2 = PAR ? hadd2u(xp, wv2[k]) : t;
                                if constexpr (TWO) {
                                    if (tap == 0 && !g.neutral) {
                                        mn[k][q][pp] = t; amn[k][q][pp] = 0u; mx[k][q][pp] = t2; amx[k][q][pp] = 0u;
                                    } else {
                                        if (tap == 0) {   // neutral padding: tap 0 may be a NaN; start from the identities
                                            mn[k][q][pp] = kPosInf2; mx[k][q][pp] = kNegInf2; amn[k][q][pp] = amx[k][q][pp] = 0u;
                                        }
                                        const unsigned ml = hbetter_mask(t, mn[k][q][pp], true);
                                        mn[k][q][pp] = hext2u(mn[k][q][pp], t, true);
                                        amn[k][q][pp] = (tap2 & ml) | (amn[k][q][pp] & ~ml);
                                        const unsigned mg = hbetter_mask(t2, mx[k][q][pp], false);
                                        mx[k][q][pp] = hext2u(mx[k][q][pp], t2, false);
                                        amx[k][q][pp] = (tap2 & mg) | (amx[k][q][pp] & ~mg);
                                    }
                                } else {
                                    if (tap == 0 && !g.neutral) {
                                        mx[k][q][pp] = t; amx[k][q][pp] = 0u;
                                    } else {
                                        if (tap == 0) { mx[k][q][pp] = TAP_MIN ? kPosInf2 : kNegInf2; amx[k][q][pp] = 0u; }
                                        const unsigned mg = hbetter_mask(t, mx[k][q][pp], TAP_MIN);
                                        mx[k][q][pp] = hext2u(mx[k][q][pp], t, TAP_MIN);
                                        amx[k][q][pp] = (tap2 & mg) | (amx[k][q][pp] & ~mg);
                                    }
                                }
                            }
                        }
                }
            } else {
                constexpr int FIRST = CARRIED ? 2 : (RS >= 3 ? 3 : RS);
                constexpr int NG = 1 + (RS - FIRST + 1) / 2;
#pragma unroll
                for (int gi = 0; gi < NG; ++gi) {
                    const int t0 = (gi == 0) ? 0 : FIRST + 2 * (gi - 1);
                    const int nt = (gi == 0) ? (FIRST < RS ? FIRST : RS) : ((RS - t0) < 2 ? (RS - t0) : 2);
                    unsigned wv[3][KPT], wv2[PAR ? 3 : 1][KPT];
#pragma unroll
                    for (int u = 0; u < 3; ++u)
                        if (u < nt) {
                            loadw<KPT>(wc + (t0 + u) * TILE_K, wv[u]);
                            if constexpr (PAR) loadw<KPT>(wc2 + (t0 + u) * TILE_K, wv2[u]);
                        }
#pragma unroll
                    for (int q = 0; q < Q; ++q)
#pragma unroll
                        for (int pp = 0; pp < 2; ++pp) {
                            unsigned xp[3];
#pragma unroll
                            for (int u = 0; u < 3; ++u)
                                if (u < nt) {
                                    const int tap = t0 + u;
                                    const int r = tap / S, sx = tap % S;
                                    if (sx == 0) xp[u] = pp == 0 ? pixel_pair<SW, EODD + 0 * SW + 0 * DW>(xw[q][r]) : pixel_pair<SW, EODD + 2 * SW + 0 * DW>(xw[q][r]);
                                    else if (sx == 1) xp[u] = pp == 0 ? pixel_pair<SW, EODD + 0 * SW + 1 * DW>(xw[q][r]) : pixel_pair<SW, EODD + 2 * SW + 1 * DW>(xw[q][r]);
                                    else xp[u] = pp == 0 ? pixel_pair<SW, EODD + 0 * SW + 2 * DW>(xw[q][r]) : pixel_pair<SW, EODD + 2 * SW + 2 * DW>(xw[q][r]);
                                }
#pragma unroll
                            for (int k = 0; k < KPT; ++k) {
                                unsigned ta[3], tb[3];
#pragma unroll
                                for (int u = 0; u < 3; ++u)
                                    if (u < nt) {
                                        ta[u] = hadd2u(xp[u], wv[u][k]);
                                        if constexpr (PAR) tb[u] = hadd2u(xp[u], wv2[u][k]);
                                    }
                                const unsigned* tm = PAR ? tb : ta;
                                if constexpr (CARRIED) {
                                    unsigned& m = best[k][q][pp];
                                    m = hext2u(m, ta[0], TAP_MIN);
                                    if (nt == 2) m = hext2u(m, ta[1], TAP_MIN);
                                } else if constexpr (TWO) {
                                    unsigned& lo = mn[k][q][pp];
                                    unsigned& hi = mx[k][q][pp];
                                    if (gi == 0) { lo = ta[0]; hi = tm[0]; }
                                    else { lo = hext2u(lo, ta[0], true); hi = hext2u(hi, tm[0], false); }
                                    if (nt >= 2) { lo = hext2u(lo, ta[1], true); hi = hext2u(hi, tm[1], false); }
                                    if (nt >= 3) { lo = hext2u(lo, ta[2], true); hi = hext2u(hi, tm[2], false); }
                                } else {
                                    unsigned& m = mx[k][q][pp];
                                    if (gi == 0) m = ta[0]; else m = hext2u(m, ta[0], TAP_MIN);
                                    if (nt >= 2) m = hext2u(m, ta[1], TAP_MIN);
                                    if (nt >= 3) m = hext2u(m, ta[2], TAP_MIN);
                                }
                            }
                        }
                }
            }

            // channel combine
            if constexpr (!CARRIED) {
                float av[KPT], bv[KPT];
                if constexpr (TWO) {
                    loadn<KPT>(as + cc * TILE_K, av);
                    loadn<KPT>(bs + cc * TILE_K, bv);
                }
#pragma unroll
                for (int k = 0; k < KPT; ++k)
#pragma unroll
                    for (int q = 0; q < Q; ++q)
#pragma unroll
                        for (int pp = 0; pp < 2; ++pp) {
                            if constexpr (TWO) {
                                fma2(av[k], bf_lo(mn[k][q][pp]), bf_hi(mn[k][q][pp]), acc[k][q][2 * pp], acc[k][q][2 * pp + 1]);
                                fma2(bv[k], bf_lo(mx[k][q][pp]), bf_hi(mx[k][q][pp]), acc[k][q][2 * pp], acc[k][q][2 * pp + 1]);
                            } else if constexpr (SUMF) {
                                addpair(bf_lo(mx[k][q][pp]), bf_hi(mx[k][q][pp]), acc[k][q][2 * pp], acc[k][q][2 * pp + 1]);
                            } else if constexpr (WIN) {
                                const unsigned m = hbetter_mask(mx[k][q][pp], best[k][q][pp], CHAN == CH_MIN);
                                best[k][q][pp] = hext2u(best[k][q][pp], mx[k][q][pp], CHAN == CH_MIN);
                                const unsigned c2 = 0x00010001u * (unsigned)c;
                                cbest[k][q][pp] = (c2 & m) | (cbest[k][q][pp] & ~m);
                            } else {
                                best[k][q][pp] = hext2u(best[k][q][pp], mx[k][q][pp], CHAN == CH_MIN);
                            }
                        }
                if constexpr (WIN && SUMF) {
                    uint8_t* codes = reinterpret_cast<uint8_t*>(p.winners);
#pragma unroll
                    for (int q = 0; q < Q; ++q) {
                        if (out_row[q] < 0) continue;
                        const int n = out_row[q] / g.OH, oh = out_row[q] - n * g.OH;
#pragma unroll
                        for (int k = 0; k < KPT; ++k) {
                            const int kk = kt * TILE_K + kg * KPT + k;
                            if (kk >= g.K) continue;
                            uint8_t* dst = codes + (((size_t)n * g.K + kk) * g.C + c) * ((size_t)g.OH * g.OWP) +
                                           (size_t)oh * g.OWP + qcol[q];
                            unsigned c01, c23;
                            if constexpr (TWO) {
                                c01 = amn[k][q][0] | (amx[k][q][0] << 4);
                                c23 = amn[k][q][1] | (amx[k][q][1] << 4);
                            } else {
                                c01 = TAP_MIN ? amx[k][q][0] : (amx[k][q][0] << 4);
                                c23 = TAP_MIN ? amx[k][q][1] : (amx[k][q][1] << 4);
                            }
                            const unsigned packed = __byte_perm(c01, c23, 0x6420);
                            // the quad's 4 codes in one store (code rows are padded to whole quads)
                            if (qcol[q] < g.OW) *reinterpret_cast<unsigned*>(dst) = packed;
                        }
                    }
                }
            }
        }
        __syncthreads();
    }

    // epilogue
    unsigned short* yg = reinterpret_cast<unsigned short*>(p.y);
    if constexpr (STATS) {
        // per-channel sums of the stored (bf16-rounded) outputs and of their squares over this tile
        static_assert(PW == 1, "one warp per channel group owns the whole pixel tile");
#pragma unroll
        for (int k = 0; k < KPT; ++k) {
            const int kk = kt * TILE_K + kg * KPT + k;
            const float bk = (p.bias && kk < g.K) ? p.bias[kk] : 0.0f;
            float s1 = 0.0f, s2 = 0.0f;
#pragma unroll
            for (int q = 0; q < Q; ++q)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float v;
                    if constexpr (SUMF) v = acc[k][q][j];
                    else v = (j & 1) ? bf_hi(best[k][q][j >> 1]) : bf_lo(best[k][q][j >> 1]);
                    if (p.bias) v = __fadd_rn(v, bk);
                    v = __bfloat162float(__float2bfloat16_rn(v));
                    if (out_row[q] >= 0 && qcol[q] + j < g.OW) { s1 += v; s2 = __fmaf_rn(v, v, s2); }
                }
#pragma unroll
            for (int dlt = 16; dlt > 0; dlt >>= 1) {
                s1 += __shfl_xor_sync(0xffffffffu, s1, dlt);
                s2 += __shfl_xor_sync(0xffffffffu, s2, dlt);
            }
            if (lane == 0 && kk < g.K)
                *reinterpret_cast<float2*>(p.stats + ((size_t)blockIdx.x * p.stats_k + kk) * 2) = make_float2(s1, s2);
        }
    }
#pragma unroll
    for (int q = 0; q < Q; ++q) {
        if (out_row[q] < 0) continue;
        const int n = out_row[q] / g.OH, oh = out_row[q] - n * g.OH;
#pragma unroll
        for (int k = 0; k < KPT; ++k) {
            const int kk = kt * TILE_K + kg * KPT + k;
            if (kk >= g.K) continue;
            const size_t o = ((size_t)n * g.K + kk) * plane + (size_t)oh * g.OW + qcol[q];
            float v[4];
            if constexpr (SUMF) {
#pragma unroll
                for (int j = 0; j < 4; ++j) v[j] = acc[k][q][j];
            } else {
                v[0] = bf_lo(best[k][q][0]); v[1] = bf_hi(best[k][q][0]);
                v[2] = bf_lo(best[k][q][1]); v[3] = bf_hi(best[k][q][1]);
            }
            if (p.bias) {
                const float bk = p.bias[kk];
#pragma unroll
                for (int j = 0; j < 4; ++j) v[j] = __fadd_rn(v[j], bk);
            }
            if (yg) {
                const __nv_bfloat162 p01 = __floats2bfloat162_rn(v[0], v[1]);
                const __nv_bfloat162 p23 = __floats2bfloat162_rn(v[2], v[3]);
                const unsigned u01 = *reinterpret_cast<const unsigned*>(&p01);
                const unsigned u23 = *reinterpret_cast<const unsigned*>(&p23);
                if (qcol[q] + 3 < g.OW && ((g.OW & 3) == 0)) {
                    *reinterpret_cast<uint2*>(yg + o) = make_uint2(u01, u23);
                } else {
                    const unsigned short e[4] = {(unsigned short)(u01 & 0xffff), (unsigned short)(u01 >> 16),
                                                 (unsigned short)(u23 & 0xffff), (unsigned short)(u23 >> 16)};
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (qcol[q] + j < g.OW) yg[o + j] = e[j];
                }
            }
            if constexpr (WIN && !SUMF) {
                int32_t* idx = reinterpret_cast<int32_t*>(p.winners);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int ow = qcol[q] + j;
                    if (ow >= g.OW) continue;
                    const unsigned cpair = cbest[k][q][j >> 1];
                    const int c = (j & 1) ? (int)(cpair >> 16) : (int)(cpair & 0xffffu);
                    const unsigned bpair = best[k][q][j >> 1];
                    const float bestv = (j & 1) ? bf_hi(bpair) : bf_lo(bpair);
                    const size_t xc = ((size_t)n * g.C + c) * chw;
                    // the window's weights in their original layout: 9 adjacent values
                    const __nv_bfloat16* wk = reinterpret_cast<const __nv_bfloat16*>(p.w) + ((size_t)kk * g.C + c) * RS;
                    int tapw = 0;
#pragma unroll
                    for (int tap = RS - 1; tap >= 0; --tap) {
                        const int ih = oh * g.sh - g.ph + (tap / S) * g.dh;
                        const int iw = ow * SW - g.pw + (tap % S) * DW;
                        const __nv_bfloat16 xv = (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W)
                                                     ? __ushort_as_bfloat16(load_x(xg, xc + (size_t)ih * g.W + iw, g.xf32))
                                                     : pad_value(g, __nv_bfloat16());
                        if (tap_add(xv, wk[tap]) == bestv) tapw = tap;
                    }
                    idx[o + j] = c * RS + tapw;
                }
            }
        }
    }
}

// PLAIN_ONLY: instantiate only the kernel without TMA and without ragged tiles (what small maps
// use); a plan that wants either is left to the caller's next choice.
template <int MODE, int CHAN, bool WIN, int R, int S, int SW, int DW, int Q, int KG, int PW, int KPT = 8,
          bool PLAIN_ONLY = false>
int launch_tiled_variant_bf16(FwdArgs& a) {
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool PAR = (MODE == TCONV_PARALLEL);
    const Geo& g = a.g;
    if (g.C > 65535) return TCONV_ERR_UNSUPPORTED;   // winner channel kept in 16 bits
    TiledPlan pl;
    pl.p.g = g;
    if (!plan_tiles<R, S, SW, DW, Q, KG, PW, KPT>(g, PAR, TWO, 2, &pl)) return TCONV_ERR_UNSUPPORTED;
    if (PLAIN_ONLY && (pl.xtma || pl.p.ragged)) return TCONV_ERR_UNSUPPORTED;
    const size_t need = pl.ws_w * (PAR ? 2 : 1) + (TWO ? 2 * pl.ws_ab : 0);
    if (!a.ws || a.ws_bytes < need) return TCONV_ERR_WORKSPACE_TOO_SMALL;
    float* wt = reinterpret_cast<float*>(a.ws);
    float* wt2 = PAR ? wt + pl.ws_w / sizeof(float) : nullptr;
    float* at = TWO ? wt + (pl.ws_w * (PAR ? 2 : 1)) / sizeof(float) : nullptr;
    float* bt = TWO ? at + pl.ws_ab / sizeof(float) : nullptr;
    CUtensorMap xmap;
    memset(&xmap, 0, sizeof(xmap));
    if (pl.xtma && !make_x_map(g, a.x, 2, pl.p, &xmap)) return TCONV_ERR_CUDA;
    const int nkt = pl.grid.y;
    const size_t nrep = (size_t)nkt * pl.p.Cpad * g.RS * pl.tile_k;
    repack_weights_bf16_kernel<0><<<(unsigned)((nrep + 255) / 256), 256, 0, a.st>>>(
        g.K, g.C, g.RS, pl.tile_k, pl.p.Cpad, nkt, (const __nv_bfloat16*)a.w, (const __nv_bfloat16*)a.w2,
        a.alpha, a.beta, (unsigned*)wt, (unsigned*)wt2, at, bt);
    pl.p.x = a.x; pl.p.w = a.w; pl.p.wt = wt; pl.p.wt2 = wt2; pl.p.at = at; pl.p.bt = bt;
    pl.p.bias = a.bias; pl.p.y = a.y; pl.p.winners = a.winners; pl.p.status = a.status;
    pl.p.stats = nullptr; pl.p.stats_k = nkt * pl.tile_k;
    if (a.stats && WIN) {
        if ((size_t)pl.grid.x * pl.p.stats_k * 2 * sizeof(float) > a.stats_bytes) return TCONV_ERR_WORKSPACE_TOO_SMALL;
        pl.p.stats = a.stats; a.stats_tiles = (int)pl.grid.x; a.stats_k = pl.p.stats_k;
    }
    pl.p.debug_drop = failure_test_switch();
#define TCONV_LAUNCH_BF16_S(XTMAV, RAGV, STATSV)                                                      \
    {                                                                                                \
        auto kern = fwd_tiled_bf16_kernel<MODE, CHAN, WIN, XTMAV, RAGV, R, S, SW, DW, Q, KG, PW, KPT, STATSV>; \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) \
            return TCONV_ERR_CUDA;                                                                   \
        kern<<<pl.grid, pl.threads, pl.smem, a.st>>>(xmap, pl.p);                                    \
    }
#define TCONV_LAUNCH_BF16(XTMAV, RAGV)                                                                \
    {                                                                                                \
        if constexpr (WIN) { if (pl.p.stats) TCONV_LAUNCH_BF16_S(XTMAV, RAGV, true) else TCONV_LAUNCH_BF16_S(XTMAV, RAGV, false) } \
        else TCONV_LAUNCH_BF16_S(XTMAV, RAGV, false)                                                 \
    }
    if constexpr (PLAIN_ONLY) {
        TCONV_LAUNCH_BF16(false, false)
        a.name = WIN ? "fwd_tiled_bf16_k4_win" : "fwd_tiled_bf16_k4";
    } else if (pl.xtma) {
        if (pl.p.ragged) TCONV_LAUNCH_BF16(true, true) else TCONV_LAUNCH_BF16(true, false)
        a.name = WIN ? "fwd_tiled_bf16_tma_win" : "fwd_tiled_bf16_tma";
    } else {
        if (pl.p.ragged) TCONV_LAUNCH_BF16(false, true) else TCONV_LAUNCH_BF16(false, false)
        a.name = WIN ? "fwd_tiled_bf16_win" : "fwd_tiled_bf16";
    }
#undef TCONV_LAUNCH_BF16
#undef TCONV_LAUNCH_BF16_S
    return TCONV_OK;
}

template <int MODE, int CHAN, bool WIN>
int launch_tiled_geom_bf16(FwdArgs& a) {
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool CARRIED = !TWO && !WIN && ((MODE == TCONV_MAX_PLUS && CHAN == CH_MAX) ||
                                              (MODE == TCONV_MIN_PLUS && CHAN == CH_MIN));
    constexpr int Q = CARRIED ? 2 : 1;
    const Geo& g = a.g;
    if (g.R == 3 && g.S == 3) {
        // Small maps with many channels at a small batch leave few warps to an SM when every thread
        // owns 8 output channels (7x7 x 512 at batch 64: 12 warps per SM, and the layer takes as long
        // as one CTA): 4 channels per thread double the warps.  Measured on the 14x14 and 7x7 layers
        // of the ResNet-18 shape at batch 64: 4 to 12 % faster with winners, 6 to 13 % slower
        // without (there the second staging of the x tiles costs more), so only with winners.
        const long warps8 = (((long)g.N * g.OH * ((g.OW + 3) / 4) + 31) / 32) * ((g.K + 7) / 8);
        const bool fine = WIN && warps8 < 148L * 32;
        if constexpr (Q == 1) {
            if (fine && g.dw == 1 && (g.sw == 1 || g.sw == 2)) {
                const int rc = g.sw == 1 ? launch_tiled_variant_bf16<MODE, CHAN, WIN, 3, 3, 1, 1, 1, 4, 1, 4, true>(a)
                                         : launch_tiled_variant_bf16<MODE, CHAN, WIN, 3, 3, 2, 1, 1, 4, 1, 4, true>(a);
                if (rc != TCONV_ERR_UNSUPPORTED) return rc;
            }
        }
        if (g.sw == 1 && g.dw == 1) return launch_tiled_variant_bf16<MODE, CHAN, WIN, 3, 3, 1, 1, Q, 4, 1>(a);
        if (g.sw == 2 && g.dw == 1) return launch_tiled_variant_bf16<MODE, CHAN, WIN, 3, 3, 2, 1, Q, 4, 1>(a);
        if (g.sw == 1 && g.dw == 2) return launch_tiled_variant_bf16<MODE, CHAN, WIN, 3, 3, 1, 2, Q, 4, 1>(a);
        if (g.sw == 1 && g.dw == 4) return launch_tiled_variant_bf16<MODE, CHAN, WIN, 3, 3, 1, 4, Q, 4, 1>(a);
    }
    // 1 x 3: the 1-D layers as signals of unit height
    if (g.R == 1 && g.S == 3 && g.sw == 1 && g.dw == 1)
        return launch_tiled_variant_bf16<MODE, CHAN, WIN, 1, 3, 1, 1, Q, 4, 1>(a);
    return TCONV_ERR_UNSUPPORTED;
}

template <int MODE, int CHAN>
int launch_fwd_tiled_bf16_inst(FwdArgs& a) {
    if (a.g.wide) return TCONV_ERR_UNSUPPORTED;
    if ((double)a.g.N * a.g.C * a.g.H * a.g.W >= 2.0e9) return TCONV_ERR_UNSUPPORTED;
    if (a.winners) return launch_tiled_geom_bf16<MODE, CHAN, true>(a);
    return launch_tiled_geom_bf16<MODE, CHAN, false>(a);
}

}  // namespace tconv

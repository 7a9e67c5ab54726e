// Backward kernels driven by the stored winners.  All are deterministic and use no
// atomics: every accumulator has exactly one writer at a time and a fixed order.
//
// Max / Min channel combine (one int32 winner per output):
//   bwd_idx_gx_kernel   a CTA owns a band of input rows of one image for every channel
//                       in shared memory; outputs are scattered tap by tap (within one tap
//                       two different output pixels never hit the same input element, and
//                       one thread walks all k of its pixel), barriers between taps.
//   bwd_idx_gw_kernel   warp-private histograms over (c, tap); lanes of a warp that hit the
//                       same bin take turns in lane order; per-CTA partials, fixed-order
//                       final sum (bwd_reduce_partials_kernel).  Also grad_bias.
// Sum channel combine (one code byte per (output, channel)):
//   bwd_code_gx_kernel  a thread owns 4 output pixels of one (n, c) and walks k, adding
//                       coef * g into its private per-tap accumulators (shared-memory
//                       columns); a gather over the taps then forms grad_x.
//   bwd_code_gw_kernel  a CTA owns one (k, c): per-tap sums of g over (n, pixel) in
//                       thread-private columns, tree-reduced; also grad_alpha / grad_beta
//                       from the branch values rebuilt as x[winner] + w[winner].
#pragma once
#include "tconv_common.cuh"

namespace tconv {

__device__ __forceinline__ unsigned lanemask_lt() {
    unsigned m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// ---------------------------------------------------------------------------------- idx: grad_x
template <typename T>
__global__ void __launch_bounds__(256)
bwd_idx_gx_kernel(Geo g, const T* __restrict__ gy, const int32_t* __restrict__ idx,
                  T* __restrict__ gx, int THI, int tiles_per_img, unsigned magic) {
    extern __shared__ float tile[];  // [C][THI][W]
    const int n = blockIdx.x / tiles_per_img;
    const int ih0 = (blockIdx.x - n * tiles_per_img) * THI;
    const int rows = min(THI, g.H - ih0);
    const int cstride = THI * g.W;
    for (int e = threadIdx.x; e < g.C * cstride; e += blockDim.x) tile[e] = 0.0f;
    __syncthreads();
    // output rows whose windows can reach the owned input rows
    const int num = ih0 + g.ph - (g.R - 1) * g.dh;
    const int oh_lo = num <= 0 ? 0 : (num + g.sh - 1) / g.sh;
    const int oh_hi = min(g.OH - 1, (ih0 + rows - 1 + g.ph) / g.sh);
    const int npix = (oh_hi - oh_lo + 1) * g.OW;
    const size_t plane = (size_t)g.OH * g.OW;
    for (int tap = 0; tap < g.RS; ++tap) {
        const int r = tap / g.S, s = tap - r * g.S;
        for (int pp = threadIdx.x; pp < npix; pp += blockDim.x) {
            const int orow = pp / g.OW;
            const int oh = oh_lo + orow, ow = pp - orow * g.OW;
            const int ih = oh * g.sh - g.ph + r * g.dh;
            const int iw = ow * g.sw - g.pw + s * g.dw;
            if (ih < ih0 || ih >= ih0 + rows || iw < 0 || iw >= g.W) continue;
            const size_t base = (size_t)n * g.K * plane + (size_t)oh * g.OW + ow;
            float* dst = tile + (ih - ih0) * g.W + iw;
#pragma unroll 4
            for (int k = 0; k < g.K; ++k) {
                const unsigned id = (unsigned)idx[base + (size_t)k * plane];
                const unsigned c = magic ? __umulhi(id, magic) : id;  // id / RS (magic 0: RS == 1)
                if ((int)(id - c * g.RS) == tap) dst[c * cstride] += to_f32(gy[base + (size_t)k * plane]);
            }
        }
        __syncthreads();
    }
    for (int e = threadIdx.x; e < g.C * rows * g.W; e += blockDim.x) {
        const int c = e / (rows * g.W);
        const int rem = e - c * rows * g.W;
        gx[((size_t)n * g.C + c) * g.H * g.W + (size_t)ih0 * g.W + rem] =
            from_f32<T>(tile[c * cstride + rem]);
    }
}

// ---------------------------------------------------------------------------------- idx: grad_w, grad_bias
template <typename T>
__global__ void __launch_bounds__(256)
bwd_idx_gw_kernel(Geo g, const T* __restrict__ gy, const int32_t* __restrict__ idx,
                  float* __restrict__ partial_w, float* __restrict__ partial_b, int n_per_chunk) {
    extern __shared__ float bins[];  // [8 warps][C*RS], then 256 floats for the bias sum
    const int CRS = g.C * g.RS;
    const int k = blockIdx.x, chunk = blockIdx.y;
    const int warp = threadIdx.x >> 5;
    float* mine = bins + warp * CRS;
    float* red = bins + 8 * CRS;
    for (int e = threadIdx.x; e < 8 * CRS; e += blockDim.x) bins[e] = 0.0f;
    __syncthreads();
    const int plane = g.OH * g.OW;
    const int n_lo = chunk * n_per_chunk, n_hi = min(g.N, n_lo + n_per_chunk);
    const unsigned lt = lanemask_lt();
    float bsum = 0.0f;
    for (int n = n_lo; n < n_hi; ++n) {
        const size_t base = ((size_t)n * g.K + k) * plane;
        for (int p0 = 0; p0 < plane; p0 += 256) {
            const int p = p0 + threadIdx.x;
            const bool valid = p < plane;
            // an out-of-range lane takes a bin of its own so that it matches nobody
            const int id = valid ? idx[base + p] : -1 - (int)threadIdx.x;
            const float gv = valid ? to_f32(gy[base + p]) : 0.0f;
            bsum += gv;
            const unsigned same = __match_any_sync(0xffffffffu, id);
            const int rank = __popc(same & lt);
            const int maxrank = __reduce_max_sync(0xffffffffu, rank);
            for (int rr = 0; rr <= maxrank; ++rr) {
                if (rank == rr && valid) mine[id] += gv;
                __syncwarp();
            }
        }
    }
    __syncthreads();
    float* out = partial_w + ((size_t)chunk * g.K + k) * CRS;
    for (int b = threadIdx.x; b < CRS; b += blockDim.x) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += bins[w * CRS + b];
        out[b] = s;
    }
    const float tb = block_sum(bsum, red);
    if (threadIdx.x == 0) partial_b[chunk * g.K + k] = tb;
}

// out[i] = sum over chunks (ascending) of partial[chunk][i]
__global__ void bwd_reduce_partials_kernel(const float* __restrict__ partial, float* __restrict__ out,
                                           size_t len, int chunks) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= len) return;
    float s = 0.0f;
    for (int c = 0; c < chunks; ++c) s += partial[(size_t)c * len + i];
    out[i] = s;
}

// ---------------------------------------------------------------------------------- codes: grad_x
struct CodeGxPlan {
    int THI, tiles_per_img;  // owned input rows per CTA
    int CB;                  // channels per CTA
    int NRmax, QPR, NQpad;   // contributing output rows (max), quads per row, padded quad count
    size_t smem;
};

// BR: 0 = both branches (compound / parallel), 1 = min branch only, 2 = max branch only.
template <typename T, int BR>
__global__ void __launch_bounds__(256)
bwd_code_gx_kernel(Geo g, const float* __restrict__ alpha, const float* __restrict__ beta,
                   const T* __restrict__ gy, const uint8_t* __restrict__ codes, T* __restrict__ gx,
                   CodeGxPlan pl) {
    extern __shared__ float A[];  // [CB][RS][4][NQpad]
    const int tile_i = blockIdx.x % pl.tiles_per_img;
    const int n = blockIdx.x / pl.tiles_per_img;
    const int c0 = blockIdx.y * pl.CB;
    const int ncb = min(pl.CB, g.C - c0);
    const int ih0 = tile_i * pl.THI;
    const int rows = min(pl.THI, g.H - ih0);
    const int num = ih0 + g.ph - (g.R - 1) * g.dh;
    const int oh_lo = num <= 0 ? 0 : (num + g.sh - 1) / g.sh;
    const int oh_hi = min(g.OH - 1, (ih0 + rows - 1 + g.ph) / g.sh);
    const int NR = oh_hi - oh_lo + 1;
    const int NQ = NR * pl.QPR;
    const int NQp = pl.NQpad;
    for (int e = threadIdx.x; e < pl.CB * g.RS * 4 * NQp; e += blockDim.x) A[e] = 0.0f;
    __syncthreads();
    const size_t plane = (size_t)g.OH * g.OW;
    const bool vec = (g.OW & 3) == 0;
    for (int q = threadIdx.x; q < NQ; q += blockDim.x) {
        const int orow = q / pl.QPR;
        const int ow0 = (q - orow * pl.QPR) * 4;
        const size_t pix = (size_t)(oh_lo + orow) * g.OW + ow0;
        float* Aq = A + q;
        for (int k = 0; k < g.K; ++k) {
            const size_t ob = ((size_t)n * g.K + k) * plane + pix;
            float gv[4];
            if (vec) {
                if constexpr (sizeof(T) == 4) {
                    const float4 v = *reinterpret_cast<const float4*>(gy + ob);
                    gv[0] = v.x; gv[1] = v.y; gv[2] = v.z; gv[3] = v.w;
                } else {
                    const uint2 v = *reinterpret_cast<const uint2*>(gy + ob);
                    gv[0] = __uint_as_float(v.x << 16); gv[1] = __uint_as_float(v.x & 0xffff0000u);
                    gv[2] = __uint_as_float(v.y << 16); gv[3] = __uint_as_float(v.y & 0xffff0000u);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) gv[j] = (ow0 + j < g.OW) ? to_f32(gy[ob + j]) : 0.0f;
            }
            for (int cb = 0; cb < ncb; ++cb) {
                const int c = c0 + cb;
                const size_t cbase = (((size_t)n * g.K + k) * g.C + c) * plane + pix;
                unsigned cw;
                if (vec) {
                    cw = *reinterpret_cast<const unsigned*>(codes + cbase);
                } else {
                    cw = 0;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (ow0 + j < g.OW) cw |= (unsigned)codes[cbase + j] << (8 * j);
                }
                float a = 1.0f, b = 1.0f;
                if constexpr (BR == 0) {
                    if (alpha) a = __ldg(alpha + (size_t)k * g.C + c);
                    if (beta) b = __ldg(beta + (size_t)k * g.C + c);
                }
                float* Ac = Aq + (size_t)cb * g.RS * 4 * NQp;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const unsigned code = (cw >> (8 * j)) & 0xffu;
                    if constexpr (BR == 0 || BR == 1) {
                        const int t = code & 15u;
                        Ac[(t * 4 + j) * NQp] += (BR == 0 ? a * gv[j] : gv[j]);
                    }
                    if constexpr (BR == 0 || BR == 2) {
                        const int t = code >> 4;
                        Ac[(t * 4 + j) * NQp] += (BR == 0 ? b * gv[j] : gv[j]);
                    }
                }
            }
        }
    }
    __syncthreads();
    // gather: every owned input element sums, over the taps, the accumulator of the output
    // pixel that reads it through that tap
    const int per_c = rows * g.W;
    for (int e = threadIdx.x; e < ncb * per_c; e += blockDim.x) {
        const int cb = e / per_c;
        const int rem = e - cb * per_c;
        const int ih = ih0 + rem / g.W, iw = rem % g.W;
        const float* Ac = A + (size_t)cb * g.RS * 4 * NQp;
        float s = 0.0f;
        for (int r = 0; r < g.R; ++r) {
            const int nh = ih + g.ph - r * g.dh;
            if (nh < 0 || nh % g.sh != 0) continue;
            const int oh = nh / g.sh;
            if (oh < oh_lo || oh > oh_hi) continue;
            for (int sx = 0; sx < g.S; ++sx) {
                const int nw = iw + g.pw - sx * g.dw;
                if (nw < 0 || nw % g.sw != 0) continue;
                const int ow = nw / g.sw;
                if (ow >= g.OW) continue;
                const int q = (oh - oh_lo) * pl.QPR + (ow >> 2);
                s += Ac[((r * g.S + sx) * 4 + (ow & 3)) * NQp + q];
            }
        }
        gx[((size_t)n * g.C + c0 + cb) * g.H * g.W + (size_t)ih * g.W + iw] = from_f32<T>(s);
    }
}

// ---------------------------------------------------------------------------------- codes: grad_w, grad_alpha, grad_beta
template <typename T, int BR>
__global__ void __launch_bounds__(256)
bwd_code_gw_kernel(Geo g, const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ w2,
                   const float* __restrict__ alpha, const float* __restrict__ beta,
                   const T* __restrict__ gy, const uint8_t* __restrict__ codes,
                   float* __restrict__ gw, float* __restrict__ gw2, float* __restrict__ galpha,
                   float* __restrict__ gbeta) {
    extern __shared__ float S[];  // [2*RS + 2][256] private columns, then tap tables
    const int c = blockIdx.x % g.C;
    const int k = blockIdx.x / g.C;
    const int tid = threadIdx.x;
    const int NB = 2 * g.RS + 2;
    float* col = S + tid;
    int* tap_dh = reinterpret_cast<int*>(S + NB * 256);
    int* tap_dw = tap_dh + g.RS;
    float* wmin_s = reinterpret_cast<float*>(tap_dw + g.RS);
    float* wmax_s = wmin_s + g.RS;
    for (int b = 0; b < NB; ++b) col[b * 256] = 0.0f;
    if (tid < g.RS) {
        tap_dh[tid] = (tid / g.S) * g.dh - g.ph;
        tap_dw[tid] = (tid % g.S) * g.dw - g.pw;
        wmin_s[tid] = to_f32(w[((size_t)k * g.C + c) * g.RS + tid]);
        wmax_s[tid] = to_f32((g.mode == TCONV_PARALLEL ? w2 : w)[((size_t)k * g.C + c) * g.RS + tid]);
    }
    __syncthreads();
    const bool need_ab = (BR == 0) && (galpha || gbeta);
    const int QPR = (g.OW + 3) >> 2;
    const int NQ = g.OH * QPR;
    const size_t plane = (size_t)g.OH * g.OW;
    const bool vec = (g.OW & 3) == 0;
    float sa = 0.0f, sb = 0.0f;
    for (int n = 0; n < g.N; ++n) {
        const T* xc = x + ((size_t)n * g.C + c) * g.H * g.W;
        const size_t obase = ((size_t)n * g.K + k) * plane;
        const size_t cbase = (((size_t)n * g.K + k) * g.C + c) * plane;
        for (int q = tid; q < NQ; q += 256) {
            const int oh = q / QPR;
            const int ow0 = (q - oh * QPR) * 4;
            const size_t pix = (size_t)oh * g.OW + ow0;
            float gv[4];
            unsigned cw;
            if (vec) {
                cw = *reinterpret_cast<const unsigned*>(codes + cbase + pix);
                if constexpr (sizeof(T) == 4) {
                    const float4 v = *reinterpret_cast<const float4*>(gy + obase + pix);
                    gv[0] = v.x; gv[1] = v.y; gv[2] = v.z; gv[3] = v.w;
                } else {
                    const uint2 v = *reinterpret_cast<const uint2*>(gy + obase + pix);
                    gv[0] = __uint_as_float(v.x << 16); gv[1] = __uint_as_float(v.x & 0xffff0000u);
                    gv[2] = __uint_as_float(v.y << 16); gv[3] = __uint_as_float(v.y & 0xffff0000u);
                }
            } else {
                cw = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool ok = ow0 + j < g.OW;
                    gv[j] = ok ? to_f32(gy[obase + pix + j]) : 0.0f;
                    if (ok) cw |= (unsigned)codes[cbase + pix + j] << (8 * j);
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (!vec && ow0 + j >= g.OW) continue;
                const unsigned code = (cw >> (8 * j)) & 0xffu;
                const int ow = ow0 + j;
                if constexpr (BR == 0 || BR == 1) {
                    const int t = code & 15u;
                    col[t * 256] += gv[j];
                    if (need_ab) {
                        const int ih = oh * g.sh + tap_dh[t], iw = ow * g.sw + tap_dw[t];
                        T xv = zero_of<T>();
                        if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) xv = xc[(size_t)ih * g.W + iw];
                        sa = __fmaf_rn(gv[j], tap_add(xv, from_f32<T>(wmin_s[t])), sa);
                    }
                }
                if constexpr (BR == 0 || BR == 2) {
                    const int t = code >> 4;
                    col[(g.RS + t) * 256] += gv[j];
                    if (need_ab) {
                        const int ih = oh * g.sh + tap_dh[t], iw = ow * g.sw + tap_dw[t];
                        T xv = zero_of<T>();
                        if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) xv = xc[(size_t)ih * g.W + iw];
                        sb = __fmaf_rn(gv[j], tap_add(xv, from_f32<T>(wmax_s[t])), sb);
                    }
                }
            }
        }
    }
    col[(2 * g.RS) * 256] = sa;
    col[(2 * g.RS + 1) * 256] = sb;
    __syncthreads();
    // fixed tree over the 256 columns of every bin
    for (int step = 128; step > 0; step >>= 1) {
        if (tid < step)
            for (int b = 0; b < NB; ++b) S[b * 256 + tid] += S[b * 256 + tid + step];
        __syncthreads();
    }
    if (tid < g.RS) {
        const float tmin = S[tid * 256], tmax = S[(g.RS + tid) * 256];
        const size_t wi = ((size_t)k * g.C + c) * g.RS + tid;
        if constexpr (BR == 0) {
            const float a = alpha ? alpha[(size_t)k * g.C + c] : 1.0f;
            const float b = beta ? beta[(size_t)k * g.C + c] : 1.0f;
            if (g.mode == TCONV_COMPOUND) {
                if (gw) gw[wi] = __fmaf_rn(a, tmin, b * tmax);
            } else {
                if (gw) gw[wi] = a * tmin;
                if (gw2) gw2[wi] = b * tmax;
            }
        } else {
            if (gw) gw[wi] = (BR == 1) ? tmin : tmax;
        }
    }
    if (BR == 0 && tid == 0) {
        if (galpha) galpha[(size_t)k * g.C + c] = S[(2 * g.RS) * 256];
        if (gbeta) gbeta[(size_t)k * g.C + c] = S[(2 * g.RS + 1) * 256];
    }
}

// ---------------------------------------------------------------------------------- host side
inline size_t bwd_ws_bytes(const Geo& g) {
    // partial histograms of the Max / Min combine: at most 16 chunks of [K][C*RS + 1] floats
    if (g.chan == CH_SUM) return 0;
    return (size_t)16 * g.K * ((size_t)g.C * g.RS + 1) * sizeof(float) + 256;
}

constexpr size_t kBwdSmemLimit = 160 * 1024;

// Plans for the winner-driven kernels; false when the shape does not fit (the caller then
// uses the any-shape kernels).
inline bool plan_idx_gx(const Geo& g, int* THI, size_t* smem) {
    const size_t row = (size_t)g.C * g.W * sizeof(float);
    if (row == 0 || row > kBwdSmemLimit) return false;
    int t = (int)(kBwdSmemLimit / row);
    if (t > g.H) t = g.H;
    // keep at least ~2 CTAs per SM worth of tiles when the batch is small
    while (t > 4 && (size_t)g.N * ((g.H + t - 1) / t) < 296) t = (t + 1) / 2;
    const int halo = (g.R - 1) * g.dh;
    if (t < g.H && t < 2 * halo) return false;  // too much redundant scanning
    *THI = t;
    *smem = row * t;
    return true;
}

inline bool plan_idx_gw(const Geo& g, int* chunks, size_t* smem) {
    const size_t bins = (size_t)8 * g.C * g.RS * sizeof(float) + 256 * sizeof(float);
    if (bins > kBwdSmemLimit) return false;
    int ch = (296 + g.K - 1) / g.K;
    if (ch > 16) ch = 16;
    if (ch > g.N) ch = g.N;
    if (ch < 1) ch = 1;
    *chunks = ch;
    *smem = bins;
    return true;
}

inline bool plan_code_gx(const Geo& g, CodeGxPlan* pl) {
    if (g.wide) return false;
    pl->QPR = (g.OW + 3) / 4;
    const int halo = (g.R - 1) * g.dh;
    for (int cb = 2; cb >= 1; --cb) {
        // rows of output quads that fit: CB * RS * 4 floats per quad
        const size_t per_quad = (size_t)cb * g.RS * 4 * sizeof(float);
        const long maxq = (long)(kBwdSmemLimit / per_quad) / 32 * 32;
        long nr = maxq / pl->QPR;
        if (nr < 1) continue;
        int thi;
        if (nr >= g.OH) {
            thi = g.H;                      // the whole image: no redundant rows
            nr = g.OH;
        } else {
            // NR = ceil((THI + halo) / sh) + 1 at most
            thi = (int)((nr - 2) * g.sh) - halo;
            if (thi < 2 * halo || thi < 1) continue;
            if (thi > g.H) thi = g.H;
        }
        pl->CB = cb;
        pl->THI = thi;
        pl->tiles_per_img = (g.H + thi - 1) / thi;
        pl->NRmax = (int)nr;
        pl->NQpad = (int)(((long)nr * pl->QPR + 31) / 32 * 32);
        pl->smem = (size_t)cb * g.RS * 4 * pl->NQpad * sizeof(float);
        if (pl->smem > kBwdSmemLimit) continue;
        return true;
    }
    return false;
}

inline size_t code_gw_smem(const Geo& g) {
    return (size_t)(2 * g.RS + 2) * 256 * sizeof(float) + (size_t)g.RS * 4 * sizeof(int);
}

}  // namespace tconv

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

// Second form of the same kernel for R*S <= 15: a thread reads the winners of its pixel once
// (batches of independent loads) and keeps only their taps, 4 bits each, in registers (blocks of
// 64 output channels).  In the phase of tap t it finds the channels whose winner is t with a few
// bit operations and touches only those: it reloads their winner (for the input channel) and
// their grad_y, the loads of the next match in flight while the current one is accumulated.
constexpr int kIdxGxKB = 8;    // output channels per staging round of bwd_idx_gx2_kernel
// RST: taps of the window when known at compile time (9: the tap loop unrolls and the targets of
// the nine phases are computed once per pixel), 0: taken from the descriptor.
template <typename T, int RST>
__global__ void __launch_bounds__(256)
bwd_idx_gx2_kernel(Geo g, const T* __restrict__ gy, const int32_t* __restrict__ idx,
                   T* __restrict__ gx, int THI, int tiles_per_img, unsigned magic) {
    constexpr int KB = kIdxGxKB;     // output channels staged per round
    constexpr int NOFF = RST > 0 ? RST : 1;
    extern __shared__ float tile[];  // [C][THI][W] | gs[KB][256] | cs[KB][256]
    const int n = blockIdx.x / tiles_per_img;
    const int ih0 = (blockIdx.x - n * tiles_per_img) * THI;
    const int rows = min(THI, g.H - ih0);
    const int cstride = THI * g.W;
    // thread-private columns: gradient and winning channel of the round's output channels
    float* gs = tile + (size_t)g.C * cstride + threadIdx.x;
    unsigned* cs = reinterpret_cast<unsigned*>(tile + (size_t)g.C * cstride + KB * 256) + threadIdx.x;
    for (int e = threadIdx.x; e < g.C * cstride; e += blockDim.x) tile[e] = 0.0f;
    const int num = ih0 + g.ph - (g.R - 1) * g.dh;
    const int oh_lo = num <= 0 ? 0 : (num + g.sh - 1) / g.sh;
    const int oh_hi = min(g.OH - 1, (ih0 + rows - 1 + g.ph) / g.sh);
    const int npix = (oh_hi - oh_lo + 1) * g.OW;
    const size_t plane = (size_t)g.OH * g.OW;
    const size_t img = (size_t)n * g.K * plane + (size_t)oh_lo * g.OW;   // first contributing pixel, k = 0
    __syncthreads();
    for (int pp0 = 0; pp0 < npix; pp0 += blockDim.x) {
        const int pp = pp0 + threadIdx.x;
        const bool live = pp < npix;
        const int orow = live ? pp / g.OW : 0;
        const int oh = oh_lo + orow, ow = live ? pp - orow * g.OW : 0;
        // element of the tile that tap t of this pixel reaches, -1 if outside the CTA's band
        auto target = [&](int tap) {
            const int r = tap / g.S, sx = tap - r * g.S;
            const int ih = oh * g.sh - g.ph + r * g.dh;
            const int iw = ow * g.sw - g.pw + sx * g.dw;
            return (live && ih >= ih0 && ih < ih0 + rows && iw >= 0 && iw < g.W) ? (ih - ih0) * g.W + iw : -1;
        };
        int off[NOFF];
        if constexpr (RST > 0) {
#pragma unroll
            for (int tap = 0; tap < RST; ++tap) off[tap] = target(tap);
        }
        const int32_t* ip = idx + img + pp;
        const T* gp = gy + img + pp;
        for (int kb0 = 0; kb0 < g.K; kb0 += KB, ip += (size_t)KB * plane, gp += (size_t)KB * plane) {
            const int kn = min(KB, g.K - kb0);
            // one round: KB winners and gradients of this pixel, all loads independent; the taps
            // stay in registers as 4-bit fields (15 marks "no channel here"), channel and gradient
            // go to the thread's shared-memory columns so that the phases below touch no global memory
            unsigned id[KB];
            float gv[KB];
#pragma unroll
            for (int i = 0; i < KB; ++i) {
                const bool ok = live && i < kn;
                id[i] = ok ? (unsigned)__ldg(ip + (size_t)i * plane) : 0xffffffffu;
                gv[i] = ok ? to_f32(__ldg(gp + (size_t)i * plane)) : 0.0f;
            }
            unsigned taps4[KB / 8];
#pragma unroll
            for (int wq = 0; wq < KB / 8; ++wq) {
                unsigned packed = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const unsigned v = id[wq * 8 + i];
                    const unsigned c = magic ? __umulhi(v, magic) : v;
                    const unsigned tap = (v == 0xffffffffu) ? 15u : (v - c * g.RS);
                    packed |= tap << (4 * i);
                    cs[(wq * 8 + i) * 256] = c;
                    gs[(wq * 8 + i) * 256] = gv[wq * 8 + i];
                }
                taps4[wq] = packed;
            }
            auto phase = [&](int tap, int o) {
                if (o >= 0) {
                    float* dst = tile + o;
                    const unsigned pat = 0x11111111u * (unsigned)tap;
#pragma unroll
                    for (int wq = 0; wq < KB / 8; ++wq) {
                        unsigned z = taps4[wq] ^ pat;       // nibble == 0 where the tap matches
                        z |= z >> 1;
                        z |= z >> 2;
                        unsigned m = ~z & 0x11111111u;      // bit 4*i set where nibble i matches
                        while (m) {
                            const int kk = wq * 8 + ((__ffs(m) - 1) >> 2);
                            m &= m - 1;
                            dst[cs[kk * 256] * cstride] += gs[kk * 256];
                        }
                    }
                }
                __syncthreads();   // inside one phase distinct pixels hit distinct inputs; phases are ordered
            };
            if constexpr (RST > 0) {
#pragma unroll
                for (int tap = 0; tap < RST; ++tap) phase(tap, off[tap]);
            } else {
                for (int tap = 0; tap < g.RS; ++tap) phase(tap, target(tap));
            }
        }
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
    // items of the chunk in a fixed order: (image, block of 256 pixels); the winners and gradients of
    // the next PF items are requested before the current ones are binned
    constexpr int PF = 4;
    const int blocks_per_img = (plane + 255) / 256;
    const int items = (n_hi - n_lo) * blocks_per_img;
    auto fetch = [&](int it, int& id, float& gv) {
        const int nn = it / blocks_per_img, p = (it - nn * blocks_per_img) * 256 + (int)threadIdx.x;
        const bool valid = it < items && p < plane;
        const size_t at = ((size_t)(n_lo + nn) * g.K + k) * plane + p;
        // an out-of-range lane takes a bin of its own so that it matches nobody
        id = valid ? __ldg(idx + at) : -1 - (int)threadIdx.x;
        gv = valid ? to_f32(__ldg(gy + at)) : 0.0f;
    };
    int idq[PF];
    float gq[PF];
#pragma unroll
    for (int u = 0; u < PF; ++u) fetch(u, idq[u], gq[u]);
    for (int it0 = 0; it0 < items; it0 += PF) {
#pragma unroll
        for (int u = 0; u < PF; ++u) {
            if (it0 + u >= items) break;
            const int id = idq[u];
            const float gv = gq[u];
            fetch(it0 + u + PF, idq[u], gq[u]);
            const bool valid = id >= 0;
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
// Most channels a CTA of bwd_code_gx_kernel handles.  One: two channels share the gradient loads,
// but the tile then takes twice the shared memory, and resident CTAs count for more (measured on
// every layer of the benchmark configurations, 3 to 27 % in favour of one channel).
constexpr int kGxCB = 1;

struct CodeGxPlan {
    int imgs;                // images per CTA (> 1 only when a CTA owns whole images of a small map)
    int THI, tiles_per_img;  // owned input rows per CTA
    int CB;                  // channels per CTA
    int NRmax, QPR, NQpad;   // contributing output rows (max), quads per row, padded quad count
    int threads;             // CTA size: 256, or more where the tile leaves room for only 1-2 CTAs per SM
    int ncblk;               // channel blocks (the fastest-varying part of the CTA index)
    int ncol, TWI, QPRt;     // column tiles of a wide map: tiles per row band, owned input columns, quads per tile row
    unsigned grid;           // CTAs: image groups x row bands x column tiles x channel blocks
    size_t smem;
};

// Loads 4 horizontally adjacent gradients (one aligned vector load: the output width these kernels
// see is a multiple of 4).
template <typename T>
__device__ __forceinline__ void load_g4(const T* p, float* gv) {
    if constexpr (sizeof(T) == 4) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(p));
        gv[0] = v.x; gv[1] = v.y; gv[2] = v.z; gv[3] = v.w;
    } else {
        const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
        gv[0] = __uint_as_float(v.x << 16); gv[1] = __uint_as_float(v.x & 0xffff0000u);
        gv[2] = __uint_as_float(v.y << 16); gv[3] = __uint_as_float(v.y & 0xffff0000u);
    }
}

// The 4 winner codes of a quad, one aligned load.  Narrow codes (R*S <= 16): one byte each, argmin
// tap in the low nibble, argmax tap in the high nibble.  WIDE (R*S <= 256): 16 bits each, argmin tap
// in the low byte, argmax tap in the high byte; `p` then points at the first of 4 adjacent codes.
template <bool WIDE> struct Codes4 { unsigned lo, hi; };
template <> struct Codes4<false> { unsigned lo; };
template <bool WIDE>
__device__ __forceinline__ Codes4<WIDE> load_codes4(const uint8_t* p) {
    Codes4<WIDE> r;
    if constexpr (!WIDE) {
        r.lo = __ldg(reinterpret_cast<const unsigned*>(p));
    } else {
        const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
        r.lo = v.x; r.hi = v.y;
    }
    return r;
}
template <bool WIDE>
__device__ __forceinline__ void taps_of(const Codes4<WIDE>& c4, int j, unsigned& tmin, unsigned& tmax) {
    if constexpr (!WIDE) {
        const unsigned code = (c4.lo >> (8 * j)) & 0xffu;
        tmin = code & 15u; tmax = code >> 4;
    } else {
        const unsigned code = ((j < 2 ? c4.lo : c4.hi) >> (16 * (j & 1))) & 0xffffu;
        tmin = code & 0xffu; tmax = code >> 8;
    }
}

// BR: 0 = both branches (compound / parallel), 1 = min branch only, 2 = max branch only.
// CB channels per CTA (the CTA's last channel block may hold fewer: those lanes idle).
// The output width is a multiple of 4 (the caller pads grad_y otherwise): aligned vector loads.
// MULTI: the CTA owns pl.imgs whole images (small maps); else one band of rows of one image.
// NTH: upper bound of the CTA size (256, or 1024 for tiles that leave room for one or two CTAs per SM).
// COLS: the band of rows is cut into pl.ncol column tiles (wide maps; never with MULTI).
template <typename T, int BR, int CB, bool MULTI, int NTH, bool WIDE, bool COLS = false>
__global__ void __launch_bounds__(NTH)
bwd_code_gx_kernel(Geo g, const float* __restrict__ alpha, const float* __restrict__ beta,
                   const T* __restrict__ gy, const uint8_t* __restrict__ codes, T* __restrict__ gx,
                   CodeGxPlan pl) {
    extern __shared__ float A[];  // [CB][RS][4][NQpad], then alpha / beta of this CTA's channels [K][CB] each
    // a CTA owns either a band of input rows of one image or pl.imgs whole images of a small map;
    // its output quads are numbered image by image
    // channel blocks vary fastest over the grid: CTAs that run together share one band of grad_y
    const int cblk = blockIdx.x % pl.ncblk;
    int xt = blockIdx.x / pl.ncblk;
    // column tile: owned input columns [iw0, iwn), first quad column qc0 of the outputs that read them
    int iw0 = 0, iwn = g.W, qc0 = 0, qpr = pl.QPR;
    if constexpr (COLS) {
        const int ct = xt % pl.ncol;
        xt /= pl.ncol;
        iw0 = ct * pl.TWI;
        iwn = min(g.W, iw0 + pl.TWI);
        const int numw = iw0 + g.pw - (g.S - 1) * g.dw;
        qc0 = (numw <= 0 ? 0 : (numw + g.sw - 1) / g.sw) >> 2;
        qpr = pl.QPRt;
    }
    const int tile_i = xt % pl.tiles_per_img;
    const int n_first = MULTI ? (xt / pl.tiles_per_img) * pl.imgs : xt / pl.tiles_per_img;
    const int nimg = MULTI ? min(pl.imgs, g.N - n_first) : 1;
    const int c0 = cblk * CB;
    const int ncb = min(CB, g.C - c0);
    const int ih0 = tile_i * pl.THI;
    const int rows = min(pl.THI, g.H - ih0);
    const int num = ih0 + g.ph - (g.R - 1) * g.dh;
    const int oh_lo = num <= 0 ? 0 : (num + g.sh - 1) / g.sh;
    const int oh_hi = min(g.OH - 1, (ih0 + rows - 1 + g.ph) / g.sh);
    const int NR = oh_hi - oh_lo + 1;
    const int NQ1 = NR * qpr;             // quads of one image (of its column tile)
    const int NQ = NQ1 * nimg;
    const int NQp = pl.NQpad;
    const int nacc = CB * g.RS * 4 * NQp;
    float* a_s = A + nacc;
    float* b_s = a_s + g.K * CB;
    for (int e = threadIdx.x; e < nacc; e += blockDim.x) A[e] = 0.0f;
    if constexpr (BR == 0) {
        for (int e = threadIdx.x; e < g.K * CB; e += blockDim.x) {
            const int k = e / CB, cb = e - k * CB;
            const bool ok = cb < ncb;
            a_s[e] = (ok && alpha) ? alpha[(size_t)k * g.C + c0 + cb] : (ok ? 1.0f : 0.0f);
            b_s[e] = (ok && beta) ? beta[(size_t)k * g.C + c0 + cb] : (ok ? 1.0f : 0.0f);
        }
    }
    __syncthreads();
    const size_t plane = (size_t)g.OH * g.OW;
    constexpr int CW = WIDE ? 2 : 1;                     // bytes per code
    const size_t cstep = (size_t)g.C * plane * CW;   // codes: one output channel k further (bytes)
    const unsigned tstride = 4u * NQp * sizeof(float); // bytes between the accumulators of two taps
    for (int q = threadIdx.x; q < NQ; q += blockDim.x) {
        const int il = MULTI ? q / NQ1 : 0;
        const int q1 = q - il * NQ1;
        const int n = n_first + il;
        const int orow = q1 / qpr;
        const int ow0 = (qc0 + q1 - orow * qpr) * 4;
        if (COLS && ow0 >= g.OW) continue;     // the last column tile's rows may end early
        const size_t pix = (size_t)(oh_lo + orow) * g.OW + ow0;
        const T* gp = gy + (size_t)n * g.K * plane + pix;
        // a channel past C reads channel C-1 again; its alpha = beta = 0 (or it is skipped below)
        const uint8_t* cp[CB];
        char* Ab[CB];
#pragma unroll
        for (int cb = 0; cb < CB; ++cb) {
            const int c = min(c0 + cb, g.C - 1);
            cp[cb] = codes + (((size_t)n * g.K * g.C + c) * plane + pix) * CW;
            Ab[cb] = reinterpret_cast<char*>(A + (size_t)cb * g.RS * 4 * NQp + q);
        }
        // operands of output channel k + PF are requested while channel k is consumed
        constexpr int PF = 4;
        float gv[PF][4];
        Codes4<WIDE> cw[PF][CB];
#pragma unroll
        for (int u = 0; u < PF; ++u)
            if (u < g.K) {
                load_g4<T>(gp + (size_t)u * plane, gv[u]);
#pragma unroll
                for (int cb = 0; cb < CB; ++cb) cw[u][cb] = load_codes4<WIDE>(cp[cb] + (size_t)u * cstep);
            }
        gp += (size_t)PF * plane;          // the next channel to request
#pragma unroll
        for (int cb = 0; cb < CB; ++cb) cp[cb] += (size_t)PF * cstep;
        for (int k0 = 0; k0 < g.K; k0 += PF) {
#pragma unroll
            for (int u = 0; u < PF; ++u) {
                const int k = k0 + u;
                if (k >= g.K) break;
#pragma unroll
                for (int cb = 0; cb < CB; ++cb) {
                    if (BR != 0 && cb >= ncb) continue;   // single-branch layers have no zero coefficient to hide behind
                    float a = 1.0f, b = 1.0f;
                    if constexpr (BR == 0) {
                        a = a_s[k * CB + cb];
                        b = b_s[k * CB + cb];
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        unsigned tmin, tmax;
                        taps_of<WIDE>(cw[u][cb], j, tmin, tmax);
                        if constexpr (BR == 0 || BR == 1) {
                            float* dst = reinterpret_cast<float*>(Ab[cb] + tmin * tstride + j * NQp * sizeof(float));
                            *dst = (BR == 0) ? __fmaf_rn(a, gv[u][j], *dst) : (*dst + gv[u][j]);
                        }
                        if constexpr (BR == 0 || BR == 2) {
                            float* dst = reinterpret_cast<float*>(Ab[cb] + tmax * tstride + j * NQp * sizeof(float));
                            *dst = (BR == 0) ? __fmaf_rn(b, gv[u][j], *dst) : (*dst + gv[u][j]);
                        }
                    }
                }
                if (k + PF < g.K) {
                    load_g4<T>(gp, gv[u]);
#pragma unroll
                    for (int cb = 0; cb < CB; ++cb) {
                        cw[u][cb] = load_codes4<WIDE>(cp[cb]);
                        cp[cb] += cstep;
                    }
                    gp += plane;
                }
            }
        }
    }
    __syncthreads();
    // gather: every owned input element sums, over the taps, the accumulator of the output
    // pixel that reads it through that tap (one warp per input row, lanes along the columns)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const bool unit_stride = (g.sh == 1 && g.sw == 1);
    for (int il = 0; il < nimg; ++il)
    for (int cb = 0; cb < ncb; ++cb) {
        const float* Ac = A + (size_t)cb * g.RS * 4 * NQp + il * NQ1;
        T* gxc = gx + ((size_t)(n_first + il) * g.C + c0 + cb) * g.H * g.W;
        for (int row = warp; row < rows; row += nwarps) {
            const int ih = ih0 + row;
            for (int iw = iw0 + lane; iw < iwn; iw += 32) {
                float s = 0.0f;
                for (int r = 0; r < g.R; ++r) {
                    int oh = ih + g.ph - r * g.dh;
                    if (!unit_stride) {
                        if (oh < 0 || oh % g.sh != 0) continue;
                        oh /= g.sh;
                    }
                    if (oh < oh_lo || oh > oh_hi) continue;
                    const float* Ar = Ac + (oh - oh_lo) * qpr - qc0;
                    for (int sx = 0; sx < g.S; ++sx) {
                        int ow = iw + g.pw - sx * g.dw;
                        if (!unit_stride) {
                            if (ow < 0 || ow % g.sw != 0) continue;
                            ow /= g.sw;
                        }
                        if (ow < 0 || ow >= g.OW) continue;
                        s += Ar[((r * g.S + sx) * 4 + (ow & 3)) * NQp + (ow >> 2)];
                    }
                }
                gxc[(size_t)ih * g.W + iw] = from_f32<T>(s);
            }
        }
    }
}

// ---------------------------------------------------------------------------------- codes: grad_w, grad_alpha, grad_beta
// One CTA per (k, c).  XS: a zero-padded copy of x (made once per backward call by
// pad_input_kernel) is available, so that the branch values x[winner] + w[winner] of
// grad_alpha / grad_beta are gathered without bounds checks.
constexpr int kGwTableInts = 2 * 16 + 2 + 4 * 16;   // per pair: tap_dh, tap_dw (RS <= 16 each, padded), two int2 tables
struct CodeGwPlan {
    int HP, WP;      // padded plane extent covering every tap of every output
    int xs_elems;    // elements of one padded plane (0: no padded copy)
    int warp;        // 1: the warp-per-pair variant of the kernel
    size_t smem;
    const void* xpad;
};

// xpad[n][c][HP][WP] = x with ph rows / pw columns of zeros in front (and zeros behind)
// TS: element type of x itself (float for a bf16 layer fed with float x: rounded here)
template <typename TS, typename T>
__global__ void pad_input_kernel(Geo g, const TS* __restrict__ x, T* __restrict__ xpad, int HP, int WP) {
    const size_t total = (size_t)g.N * g.C * HP * WP;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int pc = (int)(i % WP);
    const int pr = (int)((i / WP) % HP);
    const size_t nc = i / ((size_t)WP * HP);
    const int ih = pr - g.ph, iw = pc - g.pw;
    xpad[i] = (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) ? from_f32<T>(to_f32(x[(nc * g.H + ih) * g.W + iw])) : zero_of<T>();
}

// WARP: one warp per (k, c) pair, eight pairs per CTA, the lanes walk the pair's (image, quad)
// items and reduce with shuffles; for maps so small that a 256-thread CTA per pair would spend its
// time zeroing, synchronising and reducing.  Else one CTA per pair.
template <typename T, int BR, bool XS, bool WARP, bool WIDE>
__global__ void __launch_bounds__(256)
bwd_code_gw_kernel(Geo g, const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ w2,
                   const float* __restrict__ alpha, const float* __restrict__ beta,
                   const T* __restrict__ gy, const uint8_t* __restrict__ codes,
                   float* __restrict__ gw, float* __restrict__ gw2, float* __restrict__ galpha,
                   float* __restrict__ gbeta, CodeGwPlan pl) {
    extern __shared__ float S[];  // [2*RS + 2][256] private columns | per-tap tables (one set per pair)
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int pair = WARP ? (int)blockIdx.x * 8 + warp : (int)blockIdx.x;
    if (WARP && pair >= g.K * g.C) return;     // whole warps leave; this variant has no block barrier
    const int c = pair % g.C;
    const int k = pair / g.C;
    const int NB = 2 * g.RS + 2;
    const int me = WARP ? lane : tid;           // index of this thread among the pair's workers
    const int nworkers = WARP ? 32 : 256;
    char* colb = reinterpret_cast<char*>(S + tid);
    int* tap_dh = reinterpret_cast<int*>(S + NB * 256) + (WARP ? warp * kGwTableInts : 0);
    int* tap_dw = tap_dh + g.RS;
    // {offset of the tap inside the padded plane, weight of the tap}: min branch, max branch
    int2* tapw_min = reinterpret_cast<int2*>(tap_dw + g.RS + ((g.RS & 1) ? 0 : 0) + (((2 * g.RS) & 1) ? 1 : 0));
    int2* tapw_max = tapw_min + g.RS;
    for (int b = 0; b < NB; ++b) S[b * 256 + tid] = 0.0f;
    if (me < g.RS) {
        const int r = me / g.S, sx = me % g.S;
        tap_dh[me] = r * g.dh - g.ph;
        tap_dw[me] = sx * g.dw - g.pw;
        const size_t wi = ((size_t)k * g.C + c) * g.RS + me;
        const int off = r * g.dh * pl.WP + sx * g.dw;
        tapw_min[me] = make_int2(off, __float_as_int(to_f32(w[wi])));
        tapw_max[me] = make_int2(off, __float_as_int(to_f32((g.mode == TCONV_PARALLEL ? w2 : w)[wi])));
    }
    if constexpr (WARP) __syncwarp(); else __syncthreads();
    const bool need_ab = (BR == 0) && (galpha || gbeta);
    const int QPR = (g.OW + 3) >> 2;
    const int NQ = g.OH * QPR;
    const size_t plane = (size_t)g.OH * g.OW;
    const size_t gstep = (size_t)g.K * plane;            // grad_y: one image further
    constexpr int CW = WIDE ? 2 : 1;                      // bytes per code
    const size_t cstep = (size_t)g.K * g.C * plane * CW; // codes: one image further (bytes)
    const size_t xstep = (size_t)g.C * pl.xs_elems;      // padded x: one image further
    float sa = 0.0f, sb = 0.0f;
    // one (image, quad) item: 4 gradients gv, 4 winner codes cw, padded-x pointer xp of the item
    auto accumulate = [&](int oh, int ow0, const float* gv, const Codes4<WIDE>& cw, const T* xp) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            unsigned tmin, tmax;
            taps_of<WIDE>(cw, j, tmin, tmax);
            const float gvj = gv[j];
            if constexpr (BR == 0 || BR == 1) {
                const unsigned t = tmin;
                float* dst = reinterpret_cast<float*>(colb + t * 1024u);
                *dst += gvj;
                if (need_ab) {
                    const int2 tw = tapw_min[t];
                    T xv;
                    if constexpr (XS) {
                        xv = xp[j * g.sw + tw.x];
                    } else {
                        const int ih = oh * g.sh + tap_dh[t], iw = (ow0 + j) * g.sw + tap_dw[t];
                        xv = (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) ? xp[(size_t)ih * g.W + iw] : zero_of<T>();
                    }
                    sa = __fmaf_rn(gvj, tap_add(xv, from_f32<T>(__int_as_float(tw.y))), sa);
                }
            }
            if constexpr (BR == 0 || BR == 2) {
                const unsigned t = tmax;
                float* dst = reinterpret_cast<float*>(colb + (g.RS + t) * 1024u);
                *dst += gvj;
                if (need_ab) {
                    const int2 tw = tapw_max[t];
                    T xv;
                    if constexpr (XS) {
                        xv = xp[j * g.sw + tw.x];
                    } else {
                        const int ih = oh * g.sh + tap_dh[t], iw = (ow0 + j) * g.sw + tap_dw[t];
                        xv = (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) ? xp[(size_t)ih * g.W + iw] : zero_of<T>();
                    }
                    sb = __fmaf_rn(gvj, tap_add(xv, from_f32<T>(__int_as_float(tw.y))), sb);
                }
            }
        }
    };
    if (!WARP && NQ >= 192) {
        // large maps: a thread keeps its quad and walks the images (constant pointer strides)
        for (int q = tid; q < NQ; q += 256) {
            const int oh = q / QPR;
            const int ow0 = (q - oh * QPR) * 4;
            const size_t pix = (size_t)oh * g.OW + ow0;
            const T* gp = gy + (size_t)k * plane + pix;
            const uint8_t* cp = codes + (((size_t)k * g.C + c) * plane + pix) * CW;
            const T* xp = XS ? reinterpret_cast<const T*>(pl.xpad) + (size_t)c * pl.xs_elems +
                                   (size_t)oh * g.sh * pl.WP + ow0 * g.sw
                             : x + (size_t)c * g.H * g.W;
            float gv_cur[4], gv_nxt[4];
            Codes4<WIDE> cw_cur, cw_nxt;
            cw_nxt.lo = 0u;
            if constexpr (WIDE) cw_nxt.hi = 0u;
            load_g4<T>(gp, gv_cur);
            cw_cur = load_codes4<WIDE>(cp);
            for (int n = 0; n < g.N; ++n) {
                if (n + 1 < g.N) {
                    gp += gstep;
                    cp += cstep;
                    load_g4<T>(gp, gv_nxt);
                    cw_nxt = load_codes4<WIDE>(cp);
                }
                accumulate(oh, ow0, gv_cur, cw_cur, xp);
                xp += XS ? xstep : (size_t)g.C * g.H * g.W;
#pragma unroll
                for (int j = 0; j < 4; ++j) gv_cur[j] = gv_nxt[j];
                cw_cur = cw_nxt;
            }
        }
    } else {
        // small maps: the workers walk the flattened (image, quad) pairs with a stride of their number
        const int dn = nworkers / NQ, dq = nworkers - dn * NQ;
        int n = me / NQ, q = me - n * NQ;
        float gv_cur[4], gv_nxt[4];
        Codes4<WIDE> cw_cur, cw_nxt;
        cw_cur.lo = cw_nxt.lo = 0u;
        if constexpr (WIDE) cw_cur.hi = cw_nxt.hi = 0u;
        auto item_ptrs = [&](int n_, int q_, int& oh, int& ow0, const T*& gp, const uint8_t*& cp, const T*& xp) {
            oh = q_ / QPR;
            ow0 = (q_ - oh * QPR) * 4;
            const size_t pix = (size_t)oh * g.OW + ow0;
            gp = gy + ((size_t)n_ * g.K + k) * plane + pix;
            cp = codes + ((((size_t)n_ * g.K + k) * g.C + c) * plane + pix) * CW;
            xp = XS ? reinterpret_cast<const T*>(pl.xpad) + ((size_t)n_ * g.C + c) * pl.xs_elems +
                          (size_t)oh * g.sh * pl.WP + ow0 * g.sw
                    : x + ((size_t)n_ * g.C + c) * g.H * g.W;
        };
        int oh = 0, ow0 = 0;
        const T* gp = nullptr; const uint8_t* cp = nullptr; const T* xp = nullptr;
        bool have = n < g.N;
        if (have) {
            item_ptrs(n, q, oh, ow0, gp, cp, xp);
            load_g4<T>(gp, gv_cur);
            cw_cur = load_codes4<WIDE>(cp);
        }
        while (have) {
            int n2 = n + dn, q2 = q + dq;
            if (q2 >= NQ) { q2 -= NQ; ++n2; }
            const bool more = n2 < g.N;
            int oh2 = 0, ow2 = 0;
            const T* gp2 = nullptr; const uint8_t* cp2 = nullptr; const T* xp2 = nullptr;
            if (more) {
                item_ptrs(n2, q2, oh2, ow2, gp2, cp2, xp2);
                load_g4<T>(gp2, gv_nxt);
                cw_nxt = load_codes4<WIDE>(cp2);
            }
            accumulate(oh, ow0, gv_cur, cw_cur, xp);
            n = n2; q = q2; oh = oh2; ow0 = ow2; xp = xp2;
#pragma unroll
            for (int j = 0; j < 4; ++j) gv_cur[j] = gv_nxt[j];
            cw_cur = cw_nxt;
            have = more;
        }
    }
    float tmin = 0.0f, tmax = 0.0f, tot_a = 0.0f, tot_b = 0.0f;
    if constexpr (WARP) {
        // every bin: the 32 private values of the warp, summed by a fixed butterfly; lane t keeps
        // the totals of tap t
        for (int b = 0; b < NB; ++b) {
            float v = b < 2 * g.RS ? S[b * 256 + tid] : (b == 2 * g.RS ? sa : sb);
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
            if (b == lane) tmin = v;
            if (b == g.RS + lane) tmax = v;
            if (b == 2 * g.RS) tot_a = v;
            if (b == 2 * g.RS + 1) tot_b = v;
        }
    } else {
        S[(2 * g.RS) * 256 + tid] = sa;
        S[(2 * g.RS + 1) * 256 + tid] = sb;
        __syncthreads();
        // fixed tree over the 256 columns of every bin
        for (int step = 128; step > 0; step >>= 1) {
            if (tid < step)
                for (int b = 0; b < NB; ++b) S[b * 256 + tid] += S[b * 256 + tid + step];
            __syncthreads();
        }
        if (tid < g.RS) { tmin = S[tid * 256]; tmax = S[(g.RS + tid) * 256]; }
        tot_a = S[(2 * g.RS) * 256];
        tot_b = S[(2 * g.RS + 1) * 256];
    }
    if (me < g.RS) {
        const size_t wi = ((size_t)k * g.C + c) * g.RS + me;
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
    if (BR == 0 && me == 0) {
        if (galpha) galpha[(size_t)k * g.C + c] = tot_a;
        if (gbeta) gbeta[(size_t)k * g.C + c] = tot_b;
    }
}

// grad_bias partials: grid (K, chunks); partial[chunk][k] = sum of grad_y over the chunk's images
template <typename T>
__global__ void __launch_bounds__(256)
bwd_bias_partial_kernel(Geo g, const T* __restrict__ gy, float* __restrict__ partial, int n_per_chunk) {
    __shared__ float red[256];
    const int k = blockIdx.x, chunk = blockIdx.y;
    const size_t plane = (size_t)g.OH * g.OW;
    const int n_lo = chunk * n_per_chunk, n_hi = min(g.N, n_lo + n_per_chunk);
    float s = 0.0f;
    for (int n = n_lo; n < n_hi; ++n) {
        const T* src = gy + ((size_t)n * g.K + k) * plane;
        for (size_t j = threadIdx.x; j < plane; j += blockDim.x) s += to_f32(src[j]);
    }
    const float t = block_sum(s, red);
    if (threadIdx.x == 0) partial[chunk * g.K + k] = t;
}

// ---------------------------------------------------------------------------------- host side
inline void plan_code_gw(const Geo& g, CodeGwPlan* pl) {
    // a warp per (k, c) pair where a pair has few (image, quad) items
    pl->warp = ((size_t)g.N * g.OH * ((g.OW + 3) / 4) < 8192 && g.RS <= 16) ? 1 : 0;
    pl->smem = pl->warp ? ((size_t)(2 * g.RS + 2) * 256 + 8 * (size_t)kGwTableInts) * sizeof(float)
                        : ((size_t)(2 * g.RS + 2) * 256 + 6 * (size_t)g.RS + 4) * sizeof(float);
    pl->HP = (g.OH - 1) * g.sh + (g.R - 1) * g.dh + 1;
    pl->WP = (g.OW - 1) * g.sw + (g.S - 1) * g.dw + 1;
    if (pl->HP < g.H + g.ph) pl->HP = g.H + g.ph;   // rows / columns no output reaches still hold x
    if (pl->WP < g.W + g.pw) pl->WP = g.W + g.pw;
    pl->xs_elems = 0;
    pl->xpad = nullptr;
}
inline size_t padded_x_bytes(const Geo& g, int esize) {
    if (!two_branch(g.mode)) return 0;
    CodeGwPlan pl;
    plan_code_gw(g, &pl);
    return ((size_t)g.N * g.C * pl.HP * pl.WP * esize + 255) / 256 * 256;
}

// Sum forms whose output width is not a multiple of 4 run their code-driven kernels as a layer of
// output width OWP on a copy of grad_y with zero-padded rows (every quad whole, every load an
// aligned vector): the geometry those kernels see, and the bytes of the copy.
inline Geo widened_geo(const Geo& g) {
    Geo q = g;
    q.OW = g.OWP;
    return q;
}
inline size_t padded_gy_bytes(const Geo& g, int esize) {
    if ((g.OW & 3) == 0) return 0;
    return ((size_t)g.N * g.K * g.OH * g.OWP * esize + 255) / 256 * 256;
}

inline size_t bwd_ws_bytes(const Geo& g) {
    // partial histograms of the Max / Min combine: at most 16 chunks of [K][C*RS + 1] floats;
    // Sum forms: 16 chunks of grad_bias partials, the padded copy of x, the padded copy of grad_y
    if (g.chan == CH_SUM)
        return (size_t)16 * g.K * sizeof(float) + 256 + padded_x_bytes(widened_geo(g), 4) + padded_gy_bytes(g, 4);
    return (size_t)16 * g.K * ((size_t)g.C * g.RS + 1) * sizeof(float) + 256;
}

// grad_y with rows padded by zeros to OWP elements: one thread per padded element.
template <typename T>
__global__ void __launch_bounds__(256)
pad_grad_kernel(Geo g, const T* __restrict__ gy, T* __restrict__ out) {
    const size_t total = (size_t)g.N * g.K * g.OH * g.OWP;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int ow = (int)(i % g.OWP);
    const size_t row = i / g.OWP;
    out[i] = ow < g.OW ? gy[row * g.OW + ow] : zero_of<T>();
}

constexpr size_t kBwdSmemLimit = 160 * 1024;   // planning budget per CTA
constexpr int kBwdSmemAttr = 200 * 1024;       // opt-in ceiling set on the kernels

// Plans for the winner-driven kernels; false when the shape does not fit (the caller then
// uses the any-shape kernels).
inline bool plan_idx_gx(const Geo& g, int* THI, size_t* smem) {
    const size_t row = (size_t)g.C * g.W * sizeof(float);
    if (row == 0 || row > kBwdSmemLimit) return false;
    int t = (int)(kBwdSmemLimit / row);
    if (t > g.H) t = g.H;
    // keep at least ~2 CTAs per SM worth of tiles when the batch is small, but never bands so thin
    // that most scanned rows are halo
    const int halo = (g.R - 1) * g.dh;
    while ((t + 1) / 2 >= 2 * halo && (t + 1) / 2 >= 4 && (size_t)g.N * ((g.H + t - 1) / t) < 296) t = (t + 1) / 2;
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

// One column-tiled candidate: cb channels, ncol column tiles, budget bytes of accumulators.
inline bool plan_code_gx_cols(const Geo& g, int cb, int ncol, size_t budget, CodeGxPlan* pl) {
    const int halo = (g.R - 1) * g.dh;
    pl->QPR = (g.OW + 3) / 4;
    pl->imgs = 1;
    pl->ncol = ncol;
    pl->TWI = ((g.W + ncol - 1) / ncol + 3) / 4 * 4;
    pl->ncol = (g.W + pl->TWI - 1) / pl->TWI;
    const int span = (pl->TWI - 1 + (g.S - 1) * g.dw) / g.sw + 1;   // outputs that read one tile's columns
    pl->QPRt = (span + 3) / 4 + 1;                                   // + 1: the first of them need not start a quad
    if (pl->QPRt > pl->QPR) pl->QPRt = pl->QPR;
    const size_t per_quad = (size_t)cb * g.RS * 4 * sizeof(float);
    const long maxq = (long)(budget / per_quad) / 32 * 32;
    long nr = maxq / pl->QPRt;
    if (nr > g.OH) nr = g.OH;
    int thi = nr >= g.OH ? g.H : (int)((nr - 2) * g.sh) - halo;
    if (thi < 2 * halo || thi < 1) return false;
    if (thi > g.H) thi = g.H;
    pl->CB = cb;
    pl->THI = thi;
    pl->tiles_per_img = (g.H + thi - 1) / thi;
    pl->NRmax = (int)nr;
    pl->NQpad = (int)((nr * pl->QPRt + 31) / 32 * 32);
    pl->smem = ((size_t)cb * g.RS * 4 * pl->NQpad + 2 * (size_t)g.K * kGxCB) * sizeof(float);
    if (pl->smem > kBwdSmemLimit + 16 * 1024) return false;
    const int per_sm = (int)((227 * 1024) / (pl->smem + 1024));
    const int cap = per_sm >= 3 ? 256 : (per_sm == 2 ? 512 : 1024);
    const int nq = (int)nr * pl->QPRt;
    const int passes = (nq + cap - 1) / cap;
    int th = ((nq + passes - 1) / passes + 31) / 32 * 32;
    if (th < 256) th = 256;
    pl->threads = th < cap ? th : cap;
    if (g.wide) pl->threads = 256;
    pl->ncblk = (g.C + cb - 1) / cb;
    const size_t nct = (size_t)g.N * pl->tiles_per_img * pl->ncol * pl->ncblk;
    if (nct > 0x7fffffffu) return false;
    pl->grid = (unsigned)nct;
    return true;
}

inline bool plan_code_gx(const Geo& g, CodeGxPlan* pl) {
    pl->QPR = (g.OW + 3) / 4;
    pl->ncol = 1;
    pl->TWI = g.W;
    pl->QPRt = pl->QPR;
    // Maps with at least 128 quads (smaller ones share a CTA between several images, below): one
    // channel per CTA and a small tile, so that five CTAs stay resident per SM and hide the latency
    // of the code loads (measured on 32x32 to 128x256 maps: 5 to 35 % faster than two channels in
    // 160 KB); maps from 128 columns on are also cut into column tiles of 64 input columns, which
    // keeps the bands tall enough for their halo (128x256 at dilation 2: 20.1 -> 12.6 ms).
    if (!g.wide && (long)g.OH * pl->QPR * 2 > 256) {
        CodeGxPlan cand = *pl;
        // ... but no narrower than a CTA's 256 threads have quads for (signals of unit height)
        long ncol = (g.W + 63) / 64;
        const long most = (long)g.OH * pl->QPR / 256;
        if (ncol > most) ncol = most < 1 ? 1 : most;
        if (g.W >= 128 && plan_code_gx_cols(g, 1, (int)ncol, 72 * 1024, &cand) && cand.ncol > 1) {
            *pl = cand;
            return true;
        }
        cand = *pl;
        if (plan_code_gx_cols(g, 1, 1, 40 * 1024, &cand)) {
            *pl = cand;
            return true;
        }
    }
    const int halo = (g.R - 1) * g.dh;
    for (int cb = kGxCB; cb >= 1; --cb) {
        // rows of output quads that fit: CB * RS * 4 floats per quad
        const size_t per_quad = (size_t)cb * g.RS * 4 * sizeof(float);
        const long maxq = (long)(kBwdSmemLimit / per_quad) / 32 * 32;
        long nr = maxq / pl->QPR;
        if (nr < 1) continue;
        int thi;
        pl->imgs = 1;
        if (nr >= g.OH) {
            thi = g.H;                      // the whole image: no redundant rows
            nr = g.OH;
            // small maps: several whole images per CTA so that its 256 threads have quads to own
            const long q1 = (long)g.OH * pl->QPR;
            long im = 256 / q1;
            if (im > maxq / q1) im = maxq / q1;
            if (im > g.N) im = g.N;
            if (im > 1 && !g.wide) pl->imgs = (int)im;   // wide codes: one image per CTA (fewer kernel variants)
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
        pl->NQpad = (int)(((long)nr * pl->QPR * pl->imgs + 31) / 32 * 32);
        pl->smem = ((size_t)cb * g.RS * 4 * pl->NQpad + 2 * (size_t)g.K * kGxCB) * sizeof(float);
        if (pl->smem > kBwdSmemLimit + 16 * 1024) continue;
        // a large tile leaves one or two CTAs per SM: give them the warps the SM can hold, in
        // equal passes over the tile's quads
        const int per_sm = (int)((227 * 1024) / (pl->smem + 1024));
        int cap = per_sm >= 3 ? 256 : (per_sm == 2 ? 512 : 1024);
        const int nq = (int)nr * pl->QPR * pl->imgs;
        const int passes = (nq + cap - 1) / cap;
        int th = ((nq + passes - 1) / passes + 31) / 32 * 32;
        if (th < 256) th = 256;
        pl->threads = th < cap ? th : cap;
        if (g.wide) pl->threads = 256;
        pl->ncblk = (g.C + cb - 1) / cb;
        const size_t nct = (size_t)((g.N + pl->imgs - 1) / pl->imgs) * pl->tiles_per_img * pl->ncblk;
        if (nct > 0x7fffffffu) return false;
        pl->grid = (unsigned)nct;
        return true;
    }
    return false;
}

}  // namespace tconv

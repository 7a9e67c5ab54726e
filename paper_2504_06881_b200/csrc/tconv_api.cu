// Host side of the C ABI declared in tconv.h: descriptor validation, workspace
// accounting, kernel selection and launch.  No device memory is allocated here.
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "alu_probe.cuh"
#include "tconv_common.cuh"
#include "tconv_bwd.cuh"
#include "tconv_depthwise.cuh"
#include "tconv_generic.cuh"
#include "tconv_tiled.cuh"

using namespace tconv;

namespace tconv {
// tiled forward launchers, one per (mode, channel combine) translation unit
int fwd_inst_maxplus_sum(FwdArgs&);
int fwd_inst_maxplus_max(FwdArgs&);
int fwd_inst_maxplus_min(FwdArgs&);
int fwd_inst_minplus_sum(FwdArgs&);
int fwd_inst_minplus_max(FwdArgs&);
int fwd_inst_minplus_min(FwdArgs&);
int fwd_inst_compound(FwdArgs&);
int fwd_inst_parallel(FwdArgs&);
}  // namespace tconv

// Set non-zero by a kernel whose bounded wait on a copy gave up.
__device__ int g_tconv_device_status;

namespace {

int* device_status_ptr() {
    static int* ptrs[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_tconv_device_status) != cudaSuccess) return nullptr;
        ptrs[dev] = (int*)p;
    }
    return ptrs[dev];
}

int launch_fwd_tiled(FwdArgs& a) {
    const Geo& g = a.g;
    if (g.mode == TCONV_COMPOUND) return fwd_inst_compound(a);
    if (g.mode == TCONV_PARALLEL) return fwd_inst_parallel(a);
    if (g.mode == TCONV_MAX_PLUS)
        return g.chan == CH_MAX ? fwd_inst_maxplus_max(a)
               : g.chan == CH_MIN ? fwd_inst_maxplus_min(a) : fwd_inst_maxplus_sum(a);
    return g.chan == CH_MAX ? fwd_inst_minplus_max(a)
           : g.chan == CH_MIN ? fwd_inst_minplus_min(a) : fwd_inst_minplus_sum(a);
}

thread_local char g_last_error[256] = "";
thread_local char g_last_kernel[128] = "";
thread_local long long g_launches = 0;  // kernels launched by this thread's calls

int cuda_fail(cudaError_t e) {
    snprintf(g_last_error, sizeof(g_last_error), "%s", cudaGetErrorString(e));
    return TCONV_ERR_CUDA;
}

int check_launch() {
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? TCONV_OK : cuda_fail(e);
}

int out_extent(int in, int pad, int dil, int k, int stride) {
    const long span = (long)in + 2L * pad - (long)dil * (k - 1) - 1;
    if (span < 0) return 0;
    return (int)(span / stride) + 1;
}

// Validates the descriptor and fills the kernel-side geometry.
int make_geo(const tconv_desc_t* d, Geo* g) {
    if (!d) return TCONV_ERR_INVALID_ARG;
    if (d->N <= 0 || d->C <= 0 || d->H <= 0 || d->W <= 0 || d->K <= 0 || d->R <= 0 || d->S <= 0)
        return TCONV_ERR_INVALID_ARG;
    if (d->stride_h <= 0 || d->stride_w <= 0 || d->dil_h <= 0 || d->dil_w <= 0 || d->pad_h < 0 ||
        d->pad_w < 0)
        return TCONV_ERR_INVALID_ARG;
    if (d->mode < TCONV_MAX_PLUS || d->mode > TCONV_PARALLEL) return TCONV_ERR_INVALID_ARG;
    if (d->chan < TCONV_CHAN_DEFAULT || d->chan > TCONV_CHAN_MIN) return TCONV_ERR_INVALID_ARG;
    if (d->dtype != TCONV_F32 && d->dtype != TCONV_BF16) return TCONV_ERR_INVALID_ARG;
    if (d->pad_mode != TCONV_PAD_ZERO && d->pad_mode != TCONV_PAD_NEUTRAL) return TCONV_ERR_INVALID_ARG;
    if (d->x_dtype != TCONV_X_SAME && d->x_dtype != TCONV_X_F32) return TCONV_ERR_INVALID_ARG;
    if (d->x_dtype == TCONV_X_F32 && d->dtype != TCONV_BF16) return TCONV_ERR_INVALID_ARG;
    int chan = d->chan;
    if (chan == TCONV_CHAN_DEFAULT)
        chan = d->mode == TCONV_MAX_PLUS ? CH_MAX : d->mode == TCONV_MIN_PLUS ? CH_MIN : CH_SUM;
    if (two_branch(d->mode) && chan != CH_SUM) return TCONV_ERR_UNSUPPORTED;
    if ((long)d->R * d->S > 256) return TCONV_ERR_UNSUPPORTED;
    g->N = d->N; g->C = d->C; g->H = d->H; g->W = d->W; g->K = d->K; g->R = d->R; g->S = d->S;
    g->sh = d->stride_h; g->sw = d->stride_w; g->ph = d->pad_h; g->pw = d->pad_w;
    g->dh = d->dil_h; g->dw = d->dil_w;
    g->OH = out_extent(d->H, d->pad_h, d->dil_h, d->R, d->stride_h);
    g->OW = out_extent(d->W, d->pad_w, d->dil_w, d->S, d->stride_w);
    g->RS = d->R * d->S;
    g->OWP = (g->OW + 3) & ~3;
    g->mode = d->mode;
    g->chan = chan;
    g->wide = g->RS > 16;
    g->neutral = d->pad_mode == TCONV_PAD_NEUTRAL;
    g->xf32 = d->x_dtype == TCONV_X_F32;
    if (g->OH <= 0 || g->OW <= 0) return TCONV_ERR_INVALID_ARG;
    if (g->neutral) {
        // every window must keep a tap inside the image (else its result would be an infinity)
        auto covered = [](int out, int in, int stride, int pad, int dil, int taps) {
            for (int o = 0; o < out; ++o) {
                bool any = false;
                for (int t = 0; t < taps && !any; ++t) {
                    const long i = (long)o * stride - pad + (long)t * dil;
                    any = (i >= 0 && i < in);
                }
                if (!any) return false;
            }
            return true;
        };
        if (!covered(g->OH, g->H, g->sh, g->ph, g->dh, g->R) || !covered(g->OW, g->W, g->sw, g->pw, g->dw, g->S))
            return TCONV_ERR_UNSUPPORTED;
    }
    // one-dimensional launches index blocks with 31 bits
    const double outputs = (double)g->N * g->K * g->OH * g->OW;
    const double inputs = (double)g->N * g->C * g->H * g->W;
    if (outputs / 256 > 2.0e9 || inputs / 256 > 2.0e9 || (double)g->K * g->C * g->RS > 2.0e9)
        return TCONV_ERR_TOO_LARGE;
    return TCONV_OK;
}

size_t winner_bytes(const Geo& g) {
    if (g.chan != CH_SUM) return (size_t)g.N * g.K * g.OH * g.OW * sizeof(int32_t);
    return (size_t)g.N * g.K * g.C * g.OH * g.OWP * (g.wide ? 2 : 1);
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool misaligned(const void* p) { return p && ((uintptr_t)p & 15u) != 0; }

bool force_generic() {
    static const bool v = [] {
        const char* e = getenv("TCONV_FORCE_GENERIC");
        return e && e[0] == '1';
    }();
    return v;
}

// Upper bound of the scratch the channel statistics need: one {sum, sum of squares} pair per
// (pixel tile of the tiled kernels, output channel).  A tile holds at least one row of at most 8
// quads (32 output columns), so there are at most N * OH * ceil(quads per row / 8) of them.
size_t stats_scratch_bytes(const Geo& g) {
    const size_t tiles = (size_t)g.N * g.OH * (((g.OW + 3) / 4 + 7) / 8) + 16;
    const size_t kp = ((size_t)g.K + 63) / 64 * 64;
    return align_up(tiles * kp * 2 * sizeof(float), 256);
}

// Channel statistics from a stored output (calls without winners, layers of the any-shape kernels).
template <typename T>
void stats_from_output(const Geo& g, const void* y, float* stats_ws, float* sum_y, float* sum_y2, cudaStream_t st) {
    const int chunks = g.N < 16 ? g.N : 16, npc = (g.N + chunks - 1) / chunks;
    const int rows = (g.N + npc - 1) / npc;
    stats_direct_kernel<T><<<dim3((unsigned)g.K, (unsigned)rows), 256, 0, st>>>(g, (const T*)y, stats_ws, npc);
    stats_finish_kernel<<<(unsigned)((g.K * 32 + 255) / 256), 256, 0, st>>>(stats_ws, rows, g.K, g.K, sum_y, sum_y2);
    g_launches += 2;
}

// stats_ws: NULL, or scratch of stats_scratch_bytes() for the per-tile channel statistics, which are
// then summed into sum_y / sum_y2.
template <typename T>
int forward_t(const Geo& g, const void* x, const void* w, const void* w2, const float* alpha,
              const float* beta, const float* bias, void* y, void* winners, void* ws,
              size_t ws_bytes, cudaStream_t st, float* stats_ws = nullptr, float* sum_y = nullptr,
              float* sum_y2 = nullptr) {
    if (!force_generic()) {
        FwdArgs a;
        a.stats = stats_ws; a.stats_bytes = stats_ws ? stats_scratch_bytes(g) : 0; a.stats_tiles = 0; a.stats_k = 0;
        a.g = g; a.dtype = sizeof(T) == 4 ? TCONV_F32 : TCONV_BF16;
        a.x = x; a.w = w; a.w2 = w2; a.alpha = alpha; a.beta = beta; a.bias = bias;
        a.y = y; a.winners = winners; a.ws = ws; a.ws_bytes = ws_bytes;
        a.status = device_status_ptr(); a.st = st; a.name = "";
        const int rc = launch_fwd_tiled(a);
        if (rc == TCONV_OK) {
            snprintf(g_last_kernel, sizeof(g_last_kernel), "%s", a.name);
            g_launches += 2;  // weight repack + tiled kernel
            if (stats_ws && a.stats_tiles > 0) {
                stats_finish_kernel<<<(unsigned)((g.K * 32 + 255) / 256), 256, 0, st>>>(stats_ws, a.stats_tiles, a.stats_k,
                                                                                   g.K, sum_y, sum_y2);
                g_launches += 1;
            } else if (stats_ws) {
                stats_from_output<T>(g, y, stats_ws, sum_y, sum_y2, st);
            }
            return check_launch();
        }
        if (rc != TCONV_ERR_UNSUPPORTED) return rc;
    }
    if (g.xf32) return TCONV_ERR_UNSUPPORTED;   // float x for a bf16 layer: tiled kernels only
    const size_t total = (size_t)g.N * g.K * g.OH * g.OW;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    fwd_generic_kernel<T><<<blocks, 256, 0, st>>>(g, (const T*)x, (const T*)w, (const T*)w2, alpha,
                                                  beta, bias, (T*)y, winners);
    snprintf(g_last_kernel, sizeof(g_last_kernel), "fwd_generic");
    g_launches += 1;
    if (stats_ws && y) stats_from_output<T>(g, y, stats_ws, sum_y, sum_y2, st);
    return check_launch();
}

// grad_bias: partial sums over chunks of images at the front of the workspace, then their sum.
template <typename T>
void bias_gradient(const Geo& g, const void* gy, float* gbias, void* ws, size_t ws_bytes, bool tiled,
                   cudaStream_t st) {
    int chunks = g.N < 16 ? g.N : 16;
    if (tiled && ws && ws_bytes >= (size_t)chunks * g.K * sizeof(float)) {
        const int npc = (g.N + chunks - 1) / chunks;
        chunks = (g.N + npc - 1) / npc;
        bwd_bias_partial_kernel<T><<<dim3((unsigned)g.K, (unsigned)chunks), 256, 0, st>>>(
            g, (const T*)gy, (float*)ws, npc);
        bwd_reduce_partials_kernel<<<(unsigned)((g.K + 255) / 256), 256, 0, st>>>((const float*)ws, gbias,
                                                                               (size_t)g.K, chunks);
        g_launches += 2;
    } else {
        bwd_bias_kernel<T><<<(unsigned)g.K, 256, 0, st>>>(g, (const T*)gy, gbias);
        g_launches += 1;
    }
}

template <typename T>
int backward_sum_t(const Geo& g0, const void* x, const void* w, const void* w2, const float* alpha,
                   const float* beta, const void* gy0, const void* winners, void* gx, float* gw,
                   float* gw2, float* galpha, float* gbeta, float* gbias, void* ws, size_t ws_bytes,
                   cudaStream_t st);

template <typename T>
int backward_t(const Geo& g, const void* x, const void* w, const void* w2, const float* alpha,
               const float* beta, const void* gy, const void* winners, void* gx, float* gw,
               float* gw2, float* galpha, float* gbeta, float* gbias, void* ws, size_t ws_bytes,
               cudaStream_t st) {
    const bool twob = two_branch(g.mode);
    const bool tiled = !force_generic();
    const char* name = "bwd_generic";
    bool bias_done = false;
    if (g.chan != CH_SUM) {
        const int32_t* idx = (const int32_t*)winners;
        int thi = 0;
        size_t smem = 0;
        if (gx) {
            if (tiled && plan_idx_gx(g, &thi, &smem)) {
                const int tiles = (g.H + thi - 1) / thi;
                const unsigned magic = g.RS == 1 ? 0u : (0xFFFFFFFFu / (unsigned)g.RS) + 1u;
                if (g.RS <= 15) {
                    // the phases of this form are latency-bound: aim at three resident CTAs per SM
                    // (the tile shares the CTA's shared memory with the staging columns)
                    const size_t stage = (size_t)kIdxGxKB * 256 * 2 * sizeof(float);
                    const size_t row = (size_t)g.C * g.W * sizeof(float);
                    const int halo = (g.R - 1) * g.dh;
                    int thi2 = thi;
                    while ((row * thi2 + stage > 73 * 1024 || row * thi2 + stage > kBwdSmemAttr) &&
                           (thi2 + 1) / 2 >= 2 * halo && thi2 > 4)
                        thi2 = (thi2 + 1) / 2;
                    if (row * thi2 + stage > kBwdSmemAttr) thi2 = 0;
                    // among the band heights down to that one's half: the fewest rounds of resident
                    // CTAs times the rows a CTA scans (a band that leaves a few CTAs for a last round
                    // costs a whole round)
                    if (thi2 > 0) {
                        long best_cost = -1;
                        int best = thi2;
                        for (int t = thi2; t >= 4 && t >= 2 * halo && 2 * t >= thi2; --t) {
                            const size_t sm = row * t + stage;
                            long per_sm = (long)((227 * 1024) / (sm + 1024));
                            if (per_sm > 8) per_sm = 8;
                            if (per_sm < 1) continue;
                            const long ctas = (long)g.N * ((g.H + t - 1) / t);
                            const long rounds = (ctas + 148 * per_sm - 1) / (148 * per_sm);
                            const long cost = rounds * (t + halo);
                            if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = t; }
                        }
                        thi2 = best;
                    }
                    auto kern = g.RS == 9 ? bwd_idx_gx2_kernel<T, 9> : bwd_idx_gx2_kernel<T, 0>;
                    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemAttr) != cudaSuccess)
                        return cuda_fail(cudaGetLastError());
                    if (thi2 > 0) {
                        const int tiles2 = (g.H + thi2 - 1) / thi2;
                        kern<<<(unsigned)(g.N * tiles2), 256, (size_t)g.C * g.W * sizeof(float) * thi2 + stage, st>>>(
                            g, (const T*)gy, idx, (T*)gx, thi2, tiles2, magic);
                    } else {
                        auto kern1 = bwd_idx_gx_kernel<T>;
                        if (cudaFuncSetAttribute(kern1, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemAttr) != cudaSuccess)
                            return cuda_fail(cudaGetLastError());
                        kern1<<<(unsigned)(g.N * tiles), 256, smem, st>>>(g, (const T*)gy, idx, (T*)gx, thi, tiles, magic);
                    }
                } else {
                    auto kern = bwd_idx_gx_kernel<T>;
                    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemAttr) != cudaSuccess)
                        return cuda_fail(cudaGetLastError());
                    kern<<<(unsigned)(g.N * tiles), 256, smem, st>>>(g, (const T*)gy, idx, (T*)gx, thi, tiles, magic);
                }
                name = "bwd_idx";
            } else {
                const size_t total = (size_t)g.N * g.C * g.H * g.W;
                bwd_gx_generic_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
                    g, alpha, beta, (const T*)gy, winners, (T*)gx);
            }
            g_launches += 1;
        }
        int chunks = 0;
        if ((gw || gbias) && tiled && plan_idx_gw(g, &chunks, &smem) && ws && ws_bytes >= bwd_ws_bytes(g)) {
            const size_t CRS = (size_t)g.C * g.RS;
            float* pw = (float*)ws;
            float* pb = pw + (size_t)chunks * g.K * CRS;
            auto kern = bwd_idx_gw_kernel<T>;
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemAttr) != cudaSuccess)
                return cuda_fail(cudaGetLastError());
            const int npc = (g.N + chunks - 1) / chunks;
            kern<<<dim3((unsigned)g.K, (unsigned)chunks), 256, smem, st>>>(g, (const T*)gy, idx, pw, pb, npc);
            g_launches += 1;
            if (gw) {
                const size_t len = (size_t)g.K * CRS;
                bwd_reduce_partials_kernel<<<(unsigned)((len + 255) / 256), 256, 0, st>>>(pw, gw, len, chunks);
                g_launches += 1;
            }
            if (gbias) {
                bwd_reduce_partials_kernel<<<(unsigned)((g.K + 255) / 256), 256, 0, st>>>(pb, gbias, (size_t)g.K, chunks);
                g_launches += 1;
                bias_done = true;
            }
            name = "bwd_idx";
        } else if (gw) {
            bwd_gw_generic_kernel<T><<<(unsigned)((size_t)g.K * g.C * g.RS), 256, 0, st>>>(
                g, alpha, beta, (const T*)gy, winners, gw, gw2);
            g_launches += 1;
        }
    } else {
        return backward_sum_t<T>(g, x, w, w2, alpha, beta, gy, winners, gx, gw, gw2, galpha, gbeta, gbias, ws,
                                 ws_bytes, st);
    }
    snprintf(g_last_kernel, sizeof(g_last_kernel), "%s", name);
    if (gbias && !bias_done) bias_gradient<T>(g, gy, gbias, ws, ws_bytes, tiled, st);
    return check_launch();
}

// Backward of the Sum channel combine (layers (i), (ii), compound, parallel): per-channel winner codes.
template <typename T>
int backward_sum_t(const Geo& g0, const void* x, const void* w, const void* w2, const float* alpha,
                   const float* beta, const void* gy0, const void* winners, void* gx, float* gw,
                   float* gw2, float* galpha, float* gbeta, float* gbias, void* ws, size_t ws_bytes,
                   cudaStream_t st) {
    const bool twob = two_branch(g0.mode);
    const bool tiled = !force_generic();
    const char* name = "bwd_generic";
    // output widths that are not a multiple of 4: the code-driven kernels see a layer of width OWP
    // and a zero-padded copy of grad_y (last block of the workspace)
    Geo g = g0;
    const void* gy = gy0;
    const size_t bias_part = ((size_t)16 * g0.K * sizeof(float) + 255) / 256 * 256;
    if (tiled && (g0.OW & 3) != 0 && ws) {
        const Geo gq = widened_geo(g0);
        const size_t off = bias_part + padded_x_bytes(gq, (int)sizeof(T));
        const size_t need = padded_gy_bytes(g0, (int)sizeof(T));
        if (ws_bytes >= off + need) {
            T* gpad = (T*)((char*)ws + off);
            const size_t total = (size_t)g0.N * g0.K * g0.OH * g0.OWP;
            pad_grad_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(g0, (const T*)gy0, gpad);
            g_launches += 1;
            g = gq;
            gy = gpad;
        }
    }
    const bool quads = tiled && (g.OW & 3) == 0;   // the code-driven kernels read whole, aligned quads
    {
        const uint8_t* codes = (const uint8_t*)winners;
        const int br = twob ? 0 : (g.mode == TCONV_MIN_PLUS ? 1 : 2);
        CodeGxPlan pl;
        if (gx) {
            if (quads && plan_code_gx(g, &pl)) {
                const dim3 grid(pl.grid);
#define TCONV_GXM(BR, CBV, MULTI, NTH)                                                               \
    {                                                                                                \
        auto kern = bwd_code_gx_kernel<T, BR, CBV, MULTI, NTH, false>;                               \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemAttr) != cudaSuccess) \
            return cuda_fail(cudaGetLastError());                                                    \
        kern<<<grid, pl.threads, pl.smem, st>>>(g, alpha, beta, (const T*)gy, codes, (T*)gx, pl);   \
    }
#define TCONV_GXW(BR, CBV)                                                                           \
    {                                                                                                \
        auto kern = bwd_code_gx_kernel<T, BR, CBV, false, 256, true>;                                \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemAttr) != cudaSuccess) \
            return cuda_fail(cudaGetLastError());                                                    \
        kern<<<grid, pl.threads, pl.smem, st>>>(g, alpha, beta, (const T*)gy, codes, (T*)gx, pl);   \
    }
#define TCONV_GXC(BR, CBV, NTH)                                                                      \
    {                                                                                                \
        auto kern = bwd_code_gx_kernel<T, BR, CBV, false, NTH, false, true>;                         \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemAttr) != cudaSuccess) \
            return cuda_fail(cudaGetLastError());                                                    \
        kern<<<grid, pl.threads, pl.smem, st>>>(g, alpha, beta, (const T*)gy, codes, (T*)gx, pl);   \
    }
#define TCONV_GX(BR, CBV)                                                                            \
    {                                                                                                \
        if (pl.ncol > 1 && !g.wide) { if (pl.threads > 256) TCONV_GXC(BR, CBV, 1024) else TCONV_GXC(BR, CBV, 256) } \
        else if (g.wide) TCONV_GXW(BR, CBV)                                                          \
        else if (pl.imgs > 1) TCONV_GXM(BR, CBV, true, 256)                                          \
        else if (pl.threads > 256) TCONV_GXM(BR, CBV, false, 1024)                                   \
        else TCONV_GXM(BR, CBV, false, 256)                                                          \
    }
#define TCONV_GX2(BR) TCONV_GX(BR, 1)
                if (br == 0) TCONV_GX2(0) else if (br == 1) TCONV_GX2(1) else TCONV_GX2(2)
#undef TCONV_GX2
#undef TCONV_GX
#undef TCONV_GXM
#undef TCONV_GXW
#undef TCONV_GXC
                name = "bwd_code";
            } else {
                const size_t total = (size_t)g0.N * g0.C * g0.H * g0.W;
                bwd_gx_generic_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
                    g0, alpha, beta, (const T*)gy0, winners, (T*)gx);
            }
            g_launches += 1;
        }
        if (gw || gw2 || galpha || gbeta) {
            CodeGwPlan gp;
            plan_code_gw(g, &gp);
            if (quads && gp.smem <= kBwdSmemLimit) {
                // zero-padded copy of x for the branch values of grad_alpha / grad_beta, placed after
                // the grad_bias partials in the workspace
                const size_t pad_bytes = padded_x_bytes(g, (int)sizeof(T));
                if (br == 0 && (galpha || gbeta) && ws && ws_bytes >= bias_part + pad_bytes &&
                    (double)g.N * g.C * gp.HP * gp.WP < 2.0e9) {
                    T* xpad = (T*)((char*)ws + bias_part);
                    const size_t total = (size_t)g.N * g.C * gp.HP * gp.WP;
                    if (g.xf32) pad_input_kernel<float, T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(g, (const float*)x, xpad, gp.HP, gp.WP);
                    else pad_input_kernel<T, T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(g, (const T*)x, xpad, gp.HP, gp.WP);
                    g_launches += 1;
                    gp.xs_elems = gp.HP * gp.WP;
                    gp.xpad = xpad;
                } else if (g.xf32 && br == 0 && (galpha || gbeta)) {
                    return TCONV_ERR_UNSUPPORTED;   // float x is only read through the padded (converted) copy
                }
#define TCONV_GWK(BR, XSV, WARPV, GRID)                                                               \
    {                                                                                                \
        auto kern = bwd_code_gw_kernel<T, BR, XSV, WARPV, false>;                                    \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemAttr) != cudaSuccess) \
            return cuda_fail(cudaGetLastError());                                                    \
        kern<<<(unsigned)(GRID), 256, gp.smem, st>>>(g, (const T*)x, (const T*)w, (const T*)w2, alpha, beta, \
                                                      (const T*)gy, codes, gw, gw2, galpha, gbeta, gp); \
    }
#define TCONV_GWW(BR, XSV)                                                                           \
    {                                                                                                \
        auto kern = bwd_code_gw_kernel<T, BR, XSV, false, true>;                                     \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmemAttr) != cudaSuccess) \
            return cuda_fail(cudaGetLastError());                                                    \
        kern<<<(unsigned)((size_t)g.K * g.C), 256, gp.smem, st>>>(g, (const T*)x, (const T*)w, (const T*)w2, alpha, beta, \
                                                      (const T*)gy, codes, gw, gw2, galpha, gbeta, gp); \
    }
#define TCONV_GW(BR, XSV)                                                                            \
    {                                                                                                \
        if (g.wide) TCONV_GWW(BR, XSV)                                                               \
        else if (gp.warp) TCONV_GWK(BR, XSV, true, ((size_t)g.K * g.C + 7) / 8)                      \
        else TCONV_GWK(BR, XSV, false, (size_t)g.K * g.C)                                            \
    }
#define TCONV_GWV(BR, XSV) TCONV_GW(BR, XSV)
                if (br == 0) { if (gp.xs_elems) TCONV_GWV(0, true) else TCONV_GWV(0, false) }
                else if (br == 1) TCONV_GWV(1, false) else TCONV_GWV(2, false)
#undef TCONV_GWV
#undef TCONV_GW
#undef TCONV_GWK
#undef TCONV_GWW
                g_launches += 1;
                name = "bwd_code";
            } else {
                if (gw || gw2) {
                    bwd_gw_generic_kernel<T><<<(unsigned)((size_t)g0.K * g0.C * g0.RS), 256, 0, st>>>(
                        g0, alpha, beta, (const T*)gy0, winners, gw, gw2);
                    g_launches += 1;
                }
                if (twob && (galpha || gbeta) && g0.xf32) return TCONV_ERR_UNSUPPORTED;
                if (twob && (galpha || gbeta)) {
                    bwd_gab_generic_kernel<T><<<(unsigned)((size_t)g0.K * g0.C), 256, 0, st>>>(
                        g0, (const T*)x, (const T*)w, (const T*)w2, (const T*)gy0, winners, galpha, gbeta);
                    g_launches += 1;
                }
            }
        }
    }
    snprintf(g_last_kernel, sizeof(g_last_kernel), "%s", name);
    if (gbias) bias_gradient<T>(g0, gy0, gbias, ws, ws_bytes, tiled, st);
    return check_launch();
}

}  // namespace

// ---------------------------------------------------------------------------------- depthwise form
namespace {

// Geometry of a depthwise layer: the dense descriptor with K == C, at most 16 taps, and sizes
// whose flat indices fit 31 bits.
int make_dw_geo(const tconv_desc_t* d, Geo* g) {
    const int rc = make_geo(d, g);
    if (rc != TCONV_OK) return rc;
    if (g->K != g->C) return TCONV_ERR_INVALID_ARG;
    if (g->RS > 16 || g->neutral || g->xf32) return TCONV_ERR_UNSUPPORTED;
    g->chan = CH_SUM;
    const double lim = 2147483647.0;
    if ((double)g->N * g->C * g->OH * ((g->OW + 3) / 4) > lim || (double)g->N * g->C * g->H * g->W > lim ||
        (double)g->N * g->C * g->OH * g->OW > lim)
        return TCONV_ERR_TOO_LARGE;
    return TCONV_OK;
}

// Chunks of the per-channel reduction: enough CTAs to fill the GPU, at least 1024 items each.
int dw_chunks(const Geo& g) {
    const long items = (long)g.N * g.OH * g.OW;
    long n = (592 + g.C - 1) / g.C;
    const long most = (items + 1023) / 1024;
    if (n > most) n = most;
    if (n < 1) n = 1;
    return (int)n;
}

template <typename T>
int dw_forward_t(const Geo& g, const void* x, const void* w, const void* w2, const float* alpha,
                 const float* beta, const float* bias, void* y, void* winners, cudaStream_t st) {
    const int QPR = (g.OW + 3) / 4;
    if (g.R == 3 && g.S == 3 && g.dh == 1 && g.dw == 1 && g.sh == g.sw && (g.sw == 1 || g.sw == 2)) {
        // 3x3 windows: strips of 4 columns x 6 rows with a register window of three input rows
        const int strips = (g.OH + kDwRT - 1) / kDwRT;
        const size_t total3 = (size_t)g.N * g.C * strips * QPR;
        const unsigned blocks3 = (unsigned)((total3 + 255) / 256);
        const bool vec = (g.pw == 1 && (g.W & 3) == 0);
        // bf16 at stride 1: the same strips on packed pairs of outputs
        constexpr bool kBf16 = sizeof(T) == 2;
#define TCONV_DW3(MODE, WINV, SWV, VECV)                                                              \
    if constexpr (kBf16 && SWV == 1)                                                                  \
        dw_fwd3_bf16_kernel<MODE, WINV, VECV><<<blocks3, 256, 0, st>>>(                               \
            g, (const __nv_bfloat16*)x, (const __nv_bfloat16*)w, (const __nv_bfloat16*)w2, alpha, beta, bias, \
            (__nv_bfloat16*)y, (uint8_t*)winners, QPR, strips, (unsigned)total3);                      \
    else                                                                                              \
        dw_fwd3_kernel<T, MODE, WINV, SWV, VECV><<<blocks3, 256, 0, st>>>(                            \
            g, (const T*)x, (const T*)w, (const T*)w2, alpha, beta, bias, (T*)y, (uint8_t*)winners, QPR, strips, (unsigned)total3);
#define TCONV_DW3_V(MODE, WINV, SWV) { if (vec) TCONV_DW3(MODE, WINV, SWV, true) else TCONV_DW3(MODE, WINV, SWV, false) }
#define TCONV_DW3_S(MODE, WINV) { if (g.sw == 1) TCONV_DW3_V(MODE, WINV, 1) else TCONV_DW3_V(MODE, WINV, 2) }
#define TCONV_DW3_W(MODE) { if (winners) TCONV_DW3_S(MODE, true) else TCONV_DW3_S(MODE, false) }
        switch (g.mode) {
            case TCONV_MAX_PLUS: TCONV_DW3_W(TCONV_MAX_PLUS) break;
            case TCONV_MIN_PLUS: TCONV_DW3_W(TCONV_MIN_PLUS) break;
            case TCONV_COMPOUND: TCONV_DW3_W(TCONV_COMPOUND) break;
            default: TCONV_DW3_W(TCONV_PARALLEL) break;
        }
#undef TCONV_DW3_W
#undef TCONV_DW3_S
#undef TCONV_DW3_V
#undef TCONV_DW3
        g_launches += 1;
        snprintf(g_last_kernel, sizeof(g_last_kernel), "%s", winners ? "dw_fwd3_win" : "dw_fwd3");
        return check_launch();
    }
    const size_t total = (size_t)g.N * g.C * g.OH * QPR;
    const unsigned blocks = (unsigned)((total + 255) / 256);
#define TCONV_DW_FWD(MODE)                                                                            \
    if (winners)                                                                                     \
        dw_fwd_kernel<T, MODE, true><<<blocks, 256, 0, st>>>(g, (const T*)x, (const T*)w, (const T*)w2, alpha, beta, \
                                                             bias, (T*)y, (uint8_t*)winners, QPR, total); \
    else                                                                                             \
        dw_fwd_kernel<T, MODE, false><<<blocks, 256, 0, st>>>(g, (const T*)x, (const T*)w, (const T*)w2, alpha, beta, \
                                                              bias, (T*)y, nullptr, QPR, total);
    switch (g.mode) {
        case TCONV_MAX_PLUS: TCONV_DW_FWD(TCONV_MAX_PLUS) break;
        case TCONV_MIN_PLUS: TCONV_DW_FWD(TCONV_MIN_PLUS) break;
        case TCONV_COMPOUND: TCONV_DW_FWD(TCONV_COMPOUND) break;
        default: TCONV_DW_FWD(TCONV_PARALLEL) break;
    }
#undef TCONV_DW_FWD
    g_launches += 1;
    snprintf(g_last_kernel, sizeof(g_last_kernel), "%s", winners ? "dw_fwd_win" : "dw_fwd");
    return check_launch();
}

template <typename T>
int dw_backward_t(const Geo& g, const void* x, const void* w, const void* w2, const float* alpha,
                  const float* beta, const void* gy, const void* winners, void* gx, float* gw,
                  float* gw2, float* galpha, float* gbeta, float* gbias, void* ws, cudaStream_t st) {
    const bool twob = two_branch(g.mode), par = g.mode == TCONV_PARALLEL;
    const int br = twob ? 0 : (g.mode == TCONV_MIN_PLUS ? 1 : 2);
    const size_t wbytes = align_up((size_t)g.N * g.C * g.OH * g.OW, 256);
    const uint8_t* codes = (const uint8_t*)winners;
    float* partial = (float*)((char*)ws + wbytes);
    if (!codes) {
        // recompute the winners into the workspace (forward without an output)
        const int rc = dw_forward_t<T>(g, x, w, w2, alpha, beta, nullptr, nullptr, ws, st);
        if (rc != TCONV_OK) return rc;
        codes = (const uint8_t*)ws;
    }
    if (gx && g.R == 3 && g.S == 3 && g.dh == 1 && g.dw == 1 && g.sh == 1 && g.sw == 1) {
        // 3x3, stride 1: strips of 4 input columns x 6 input rows over a register window
        const int QPRI = (g.W + 3) / 4, strips = (g.H + 5) / 6;
        const size_t total = (size_t)g.N * g.C * strips * QPRI;
        const unsigned blocks = (unsigned)((total + 255) / 256);
        const bool vec = (g.pw == 1 && (g.OW & 3) == 0);
#define TCONV_DW_GX3(BR, VECV)                                                                        \
    dw_bwd_gx3_kernel<T, BR, VECV><<<blocks, 256, 0, st>>>(g, alpha, beta, (const T*)gy, codes, (T*)gx, QPRI, strips, \
                                                           (unsigned)total);
#define TCONV_DW_GX3_V(BR) { if (vec) TCONV_DW_GX3(BR, true) else TCONV_DW_GX3(BR, false) }
        if (br == 0) TCONV_DW_GX3_V(0) else if (br == 1) TCONV_DW_GX3_V(1) else TCONV_DW_GX3_V(2)
#undef TCONV_DW_GX3_V
#undef TCONV_DW_GX3
        g_launches += 1;
    } else if (gx && g.R == 3 && g.S == 3 && g.dh == 1 && g.dw == 1 && g.sh == 2 && g.sw == 2 && g.ph == 1 && g.pw == 1) {
        // 3x3, stride 2, padding 1: one thread per 2 x 2 input block
        const int HB = (g.H + 1) / 2, WB = (g.W + 1) / 2;
        const size_t total = (size_t)g.N * g.C * HB * WB;
        const unsigned blocks = (unsigned)((total + 255) / 256);
        if (br == 0) dw_bwd_gx_s2_kernel<T, 0><<<blocks, 256, 0, st>>>(g, alpha, beta, (const T*)gy, codes, (T*)gx, HB, WB, (unsigned)total);
        else if (br == 1) dw_bwd_gx_s2_kernel<T, 1><<<blocks, 256, 0, st>>>(g, alpha, beta, (const T*)gy, codes, (T*)gx, HB, WB, (unsigned)total);
        else dw_bwd_gx_s2_kernel<T, 2><<<blocks, 256, 0, st>>>(g, alpha, beta, (const T*)gy, codes, (T*)gx, HB, WB, (unsigned)total);
        g_launches += 1;
    } else if (gx) {
        const size_t total = (size_t)g.N * g.C * g.H * g.W;
        const unsigned blocks = (unsigned)((total + 255) / 256);
#define TCONV_DW_GX(BR, STV) dw_bwd_gx_kernel<T, BR, STV><<<blocks, 256, 0, st>>>(g, alpha, beta, (const T*)gy, codes, (T*)gx, total);
#define TCONV_DW_GX_S(BR) { if (g.sh == 2 && g.sw == 2) TCONV_DW_GX(BR, 2) else TCONV_DW_GX(BR, 0) }
        if (br == 0) TCONV_DW_GX_S(0) else if (br == 1) TCONV_DW_GX_S(1) else TCONV_DW_GX_S(2)
#undef TCONV_DW_GX_S
#undef TCONV_DW_GX
        g_launches += 1;
    }
    if (gw || gw2 || galpha || gbeta || gbias) {
        const int nch = dw_chunks(g);
        const dim3 grid((unsigned)g.C, (unsigned)nch);
        const size_t smem = (size_t)kDwAcc * 256 * sizeof(float);
        const int need_ab = (twob && (galpha || gbeta)) ? 1 : 0;
#define TCONV_DW_PAR(BR, PARV)                                                                        \
    {                                                                                                \
        auto kern = dw_bwd_params_kernel<T, BR, PARV>;                                               \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) \
            return cuda_fail(cudaGetLastError());                                                    \
        kern<<<grid, 256, smem, st>>>(g, (const T*)x, (const T*)w, (const T*)w2, (const T*)gy, codes, partial, nch, need_ab); \
    }
        const bool k3 = g.R == 3 && g.S == 3 && g.dh == 1 && g.dw == 1 && g.sh == g.sw && (g.sw == 1 || g.sw == 2) &&
                        nch <= g.N && g.OH * g.OW >= 100;   // tiny planes: too few strips per image
        if (k3) {
            // 3x3 windows: strips over a register window, the chunks are ranges of images
            const int QPR3 = (g.OW + 3) / 4, strips3 = (g.OH + kDwRT - 1) / kDwRT;
            const bool vec3 = (g.pw == 1 && (g.W & 3) == 0);
#define TCONV_DW_P3(BR, PARV, SWV, VECV)                                                              \
    {                                                                                                \
        auto kern = dw_bwd_params3_kernel<T, BR, PARV, SWV, VECV>;                                   \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) \
            return cuda_fail(cudaGetLastError());                                                    \
        kern<<<grid, 256, smem, st>>>(g, (const T*)x, (const T*)w, (const T*)w2, (const T*)gy, codes, partial, nch, \
                                      need_ab, QPR3, strips3);                                       \
    }
#define TCONV_DW_P3V(BR, PARV, SWV) { if (vec3) TCONV_DW_P3(BR, PARV, SWV, true) else TCONV_DW_P3(BR, PARV, SWV, false) }
#define TCONV_DW_P3S(BR, PARV) { if (g.sw == 1) TCONV_DW_P3V(BR, PARV, 1) else TCONV_DW_P3V(BR, PARV, 2) }
            if (br == 0) { if (par) TCONV_DW_P3S(0, true) else TCONV_DW_P3S(0, false) }
            else if (br == 1) TCONV_DW_P3S(1, false)
            else TCONV_DW_P3S(2, false)
#undef TCONV_DW_P3S
#undef TCONV_DW_P3V
#undef TCONV_DW_P3
        } else if (br == 0) { if (par) TCONV_DW_PAR(0, true) else TCONV_DW_PAR(0, false) }
        else if (br == 1) TCONV_DW_PAR(1, false)
        else TCONV_DW_PAR(2, false)
#undef TCONV_DW_PAR
        const int n = g.C * kDwAcc;
        dw_bwd_finish_kernel<<<(n + 255) / 256, 256, 0, st>>>(g, partial, nch, g.mode, alpha, beta, gw, gw2, galpha,
                                                             gbeta, gbias);
        g_launches += 2;
    }
    snprintf(g_last_kernel, sizeof(g_last_kernel), "%s", "dw_bwd");
    return check_launch();
}

}  // namespace

extern "C" {

int tconv_output_shape(const tconv_desc_t* desc, int32_t* OH, int32_t* OW) {
    Geo g;
    const int rc = make_geo(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (OH) *OH = g.OH;
    if (OW) *OW = g.OW;
    return TCONV_OK;
}

size_t tconv_winner_bytes(const tconv_desc_t* desc) {
    Geo g;
    if (make_geo(desc, &g) != TCONV_OK) return 0;
    return winner_bytes(g);
}

size_t tconv_workspace_bytes(const tconv_desc_t* desc, int backward) {
    Geo g;
    if (make_geo(desc, &g) != TCONV_OK) return 0;
    const size_t fwd = align_up(tiled_ws_bytes(g), 256);  // repacked weights, alpha, beta
    if (!backward) return fwd;
    // winners recomputed (by a forward pass) into the workspace when the caller passes none;
    // the forward scratch and the backward partial sums are not live at the same time
    const size_t bwd = align_up(bwd_ws_bytes(g), 256);
    return align_up(winner_bytes(g), 256) + (fwd > bwd ? fwd : bwd);
}

int tconv_forward(const tconv_desc_t* desc, const void* x, const void* w, const void* w2,
                  const float* alpha, const float* beta, const float* bias, void* y, void* winners,
                  void* workspace, size_t workspace_bytes, void* stream) {
    Geo g;
    int rc = make_geo(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (!x || !w || !y) return TCONV_ERR_INVALID_ARG;
    if (g.mode == TCONV_PARALLEL && !w2) return TCONV_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(w) || misaligned(w2) || misaligned(alpha) || misaligned(beta) ||
        misaligned(bias) || misaligned(y) || misaligned(winners) || misaligned(workspace))
        return TCONV_ERR_MISALIGNED;
    if (workspace_bytes < tconv_workspace_bytes(desc, 0)) return TCONV_ERR_WORKSPACE_TOO_SMALL;
    if (!two_branch(g.mode)) { alpha = nullptr; beta = nullptr; }
    cudaStream_t st = (cudaStream_t)stream;
    g_last_error[0] = 0;
    if (desc->dtype == TCONV_F32)
        return forward_t<float>(g, x, w, w2, alpha, beta, bias, y, winners, workspace,
                                workspace_bytes, st);
    return forward_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, bias, y, winners, workspace,
                                    workspace_bytes, st);
}

size_t tconv_stats_workspace_bytes(const tconv_desc_t* desc) {
    Geo g;
    if (make_geo(desc, &g) != TCONV_OK) return 0;
    return tconv_workspace_bytes(desc, 0) + stats_scratch_bytes(g);
}

int tconv_forward_stats(const tconv_desc_t* desc, const void* x, const void* w, const void* w2,
                        const float* alpha, const float* beta, const float* bias, void* y, void* winners,
                        float* sum_y, float* sum_y2, void* workspace, size_t workspace_bytes, void* stream) {
    Geo g;
    int rc = make_geo(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (!x || !w || !y || !sum_y || !sum_y2 || !workspace) return TCONV_ERR_INVALID_ARG;
    if (g.mode == TCONV_PARALLEL && !w2) return TCONV_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(w) || misaligned(w2) || misaligned(alpha) || misaligned(beta) ||
        misaligned(bias) || misaligned(y) || misaligned(winners) || misaligned(workspace) || misaligned(sum_y) ||
        misaligned(sum_y2))
        return TCONV_ERR_MISALIGNED;
    const size_t fwd = tconv_workspace_bytes(desc, 0);
    if (workspace_bytes < fwd + stats_scratch_bytes(g)) return TCONV_ERR_WORKSPACE_TOO_SMALL;
    if (!two_branch(g.mode)) { alpha = nullptr; beta = nullptr; }
    cudaStream_t st = (cudaStream_t)stream;
    g_last_error[0] = 0;
    float* stats_ws = (float*)((char*)workspace + fwd);
    if (desc->dtype == TCONV_F32)
        return forward_t<float>(g, x, w, w2, alpha, beta, bias, y, winners, workspace, fwd, st, stats_ws, sum_y, sum_y2);
    return forward_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, bias, y, winners, workspace, fwd, st, stats_ws, sum_y,
                                    sum_y2);
}

int tconv_backward(const tconv_desc_t* desc, const void* x, const void* w, const void* w2,
                   const float* alpha, const float* beta, const void* grad_y, const void* winners,
                   void* grad_x, float* grad_w, float* grad_w2, float* grad_alpha,
                   float* grad_beta, float* grad_bias, void* workspace, size_t workspace_bytes,
                   void* stream) {
    Geo g;
    int rc = make_geo(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (!x || !w || !grad_y) return TCONV_ERR_INVALID_ARG;
    if (g.mode == TCONV_PARALLEL && !w2) return TCONV_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(w) || misaligned(w2) || misaligned(alpha) || misaligned(beta) ||
        misaligned(grad_y) || misaligned(winners) || misaligned(grad_x) || misaligned(grad_w) ||
        misaligned(grad_w2) || misaligned(grad_alpha) || misaligned(grad_beta) ||
        misaligned(grad_bias) || misaligned(workspace))
        return TCONV_ERR_MISALIGNED;
    if (!two_branch(g.mode)) { alpha = nullptr; beta = nullptr; grad_alpha = nullptr; grad_beta = nullptr; }
    if (g.mode != TCONV_PARALLEL) grad_w2 = nullptr;
    cudaStream_t st = (cudaStream_t)stream;
    g_last_error[0] = 0;
    char* ws = (char*)workspace;
    size_t ws_left = workspace_bytes;
    if (!winners) {
        // recompute the winners with a forward pass that stores winners only
        // (the kernels accept y == NULL internally)
        const size_t wb = align_up(winner_bytes(g), 256);
        if (!ws || ws_left < wb) return TCONV_ERR_WORKSPACE_TOO_SMALL;
        void* wbuf = ws;
        ws += wb;
        ws_left -= wb;
        rc = (desc->dtype == TCONV_F32)
                 ? forward_t<float>(g, x, w, w2, alpha, beta, nullptr, nullptr, wbuf, ws, ws_left, st)
                 : forward_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, nullptr, nullptr, wbuf, ws,
                                            ws_left, st);
        if (rc != TCONV_OK) return rc;
        winners = wbuf;
    }
    if (desc->dtype == TCONV_F32)
        return backward_t<float>(g, x, w, w2, alpha, beta, grad_y, winners, grad_x, grad_w, grad_w2,
                                 grad_alpha, grad_beta, grad_bias, ws, ws_left, st);
    return backward_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, grad_y, winners, grad_x, grad_w,
                                     grad_w2, grad_alpha, grad_beta, grad_bias, ws, ws_left, st);
}

double tconv_paper_ops(const tconv_desc_t* desc) {
    Geo g;
    if (make_geo(desc, &g) != TCONV_OK) return 0.0;
    const double P = (double)g.N * g.K * g.OH * g.OW, C = g.C, RS = g.RS;
    if (g.mode == TCONV_COMPOUND) return ((RS * C + 2 * C - 1) + 2 * (RS - 1) * C + 2 * C) * P;
    if (g.mode == TCONV_PARALLEL) return ((2 * RS * C + 2 * C - 1) + 2 * (RS - 1) * C + 2 * C) * P;
    if (g.chan == CH_SUM) return ((C - 1 + RS * C) + (RS - 1) * C) * P;
    return (RS * C + (RS * C - 1)) * P;
}

// ---------------------------------------------------------------------------------- depthwise form
size_t tconv_dw_winner_bytes(const tconv_desc_t* desc) {
    Geo g;
    if (make_dw_geo(desc, &g) != TCONV_OK) return 0;
    return (size_t)g.N * g.C * g.OH * g.OW;
}

size_t tconv_dw_workspace_bytes(const tconv_desc_t* desc, int backward) {
    Geo g;
    if (make_dw_geo(desc, &g) != TCONV_OK || !backward) return 0;
    return align_up((size_t)g.N * g.C * g.OH * g.OW, 256) + (size_t)dw_chunks(g) * g.C * kDwAcc * sizeof(float) + 256;
}

int tconv_dw_forward(const tconv_desc_t* desc, const void* x, const void* w, const void* w2,
                     const float* alpha, const float* beta, const float* bias, void* y, void* winners,
                     void* stream) {
    g_last_error[0] = 0;
    Geo g;
    const int rc = make_dw_geo(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (!x || !w || (!y && !winners)) return TCONV_ERR_INVALID_ARG;
    if (g.mode == TCONV_PARALLEL && !w2) return TCONV_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(y) || misaligned(winners)) return TCONV_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    return desc->dtype == TCONV_F32
               ? dw_forward_t<float>(g, x, w, w2, alpha, beta, bias, y, winners, st)
               : dw_forward_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, bias, y, winners, st);
}

int tconv_dw_backward(const tconv_desc_t* desc, const void* x, const void* w, const void* w2,
                      const float* alpha, const float* beta, const void* grad_y, const void* winners,
                      void* grad_x, float* grad_w, float* grad_w2, float* grad_alpha, float* grad_beta,
                      float* grad_bias, void* workspace, size_t workspace_bytes, void* stream) {
    g_last_error[0] = 0;
    Geo g;
    const int rc = make_dw_geo(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (!x || !w || !grad_y) return TCONV_ERR_INVALID_ARG;
    if (g.mode == TCONV_PARALLEL && !w2) return TCONV_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(grad_y) || misaligned(winners) || misaligned(grad_x) || misaligned(workspace))
        return TCONV_ERR_MISALIGNED;
    if (!workspace || workspace_bytes < tconv_dw_workspace_bytes(desc, 1)) return TCONV_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    return desc->dtype == TCONV_F32
               ? dw_backward_t<float>(g, x, w, w2, alpha, beta, grad_y, winners, grad_x, grad_w, grad_w2,
                                      grad_alpha, grad_beta, grad_bias, workspace, st)
               : dw_backward_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, grad_y, winners, grad_x, grad_w,
                                              grad_w2, grad_alpha, grad_beta, grad_bias, workspace, st);
}

int tconv_alu_probe(int variant, int iters, void* sink, double* taps_per_launch, void* stream) {
    // variants PROBE_COUNT .. 2 * PROBE_COUNT - 1: the same mixes with operand feedback
    if (variant < 0 || variant >= 2 * PROBE_COUNT || iters <= 0 || !sink) return TCONV_ERR_INVALID_ARG;
    const bool feed = variant >= PROBE_COUNT;
    const int mix = feed ? variant - PROBE_COUNT : variant;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    const unsigned blocks = (unsigned)sms * 8u;
    cudaStream_t st = (cudaStream_t)stream;
    const float seed = 1.0009765625f;
#define TCONV_PROBE_CASE(V)                                                                          \
    case V:                                                                                          \
        if (feed) alu_probe_kernel<V, true><<<blocks, 256, 0, st>>>(iters, seed, (float*)sink);      \
        else alu_probe_kernel<V, false><<<blocks, 256, 0, st>>>(iters, seed, (float*)sink);          \
        break;
    switch (mix) {
        TCONV_PROBE_CASE(0) TCONV_PROBE_CASE(1) TCONV_PROBE_CASE(2) TCONV_PROBE_CASE(3)
        TCONV_PROBE_CASE(4) TCONV_PROBE_CASE(5) TCONV_PROBE_CASE(6) TCONV_PROBE_CASE(7)
        TCONV_PROBE_CASE(8) TCONV_PROBE_CASE(9) TCONV_PROBE_CASE(10) TCONV_PROBE_CASE(11)
        TCONV_PROBE_CASE(12) TCONV_PROBE_CASE(13) TCONV_PROBE_CASE(14) TCONV_PROBE_CASE(15)
        TCONV_PROBE_CASE(16) TCONV_PROBE_CASE(17) TCONV_PROBE_CASE(18) TCONV_PROBE_CASE(19)
        TCONV_PROBE_CASE(20) TCONV_PROBE_CASE(21) TCONV_PROBE_CASE(22) TCONV_PROBE_CASE(23)
    }
#undef TCONV_PROBE_CASE
    static_assert(PROBE_COUNT == 24, "one case per probe variant");
    g_launches += 1;
    if (taps_per_launch)
        *taps_per_launch = (double)blocks * 256.0 * iters * probe_taps_per_iter(mix);
    return check_launch();
}

const char* tconv_alu_probe_name(int variant) {
    static char names[2 * PROBE_COUNT][40];
    if (variant < 0 || variant >= 2 * PROBE_COUNT) return nullptr;
    if (variant < PROBE_COUNT) return kProbeNames[variant];
    snprintf(names[variant], sizeof(names[variant]), "%s_fb", kProbeNames[variant - PROBE_COUNT]);
    return names[variant];
}

const char* tconv_status_string(int status) {
    switch (status) {
        case TCONV_OK: return "ok";
        case TCONV_ERR_INVALID_ARG: return "invalid argument";
        case TCONV_ERR_UNSUPPORTED: return "unsupported descriptor";
        case TCONV_ERR_MISALIGNED: return "pointer not 16-byte aligned";
        case TCONV_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case TCONV_ERR_CUDA: return "CUDA error";
        case TCONV_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case TCONV_ERR_TOO_LARGE: return "size too large";
        default: return "unknown status";
    }
}

int tconv_device_status(void* stream) {
    int* p = device_status_ptr();
    if (!p) return cuda_fail(cudaGetLastError());
    cudaStream_t st = (cudaStream_t)stream;
    int v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, p, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    if (v == 0) return TCONV_OK;
    e = cudaMemsetAsync(p, 0, sizeof(int), st);
    if (e != cudaSuccess) return cuda_fail(e);
    return TCONV_ERR_DEVICE_TIMEOUT;
}

// ---- forward pass for callers that cannot allocate device memory --------------------
// Scratch of the allocation-free entry point: lives in the library image, so every GPU
// that loads the library holds these bytes until the process exits.
#define TCONV_NOALLOC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_noalloc_scratch[TCONV_NOALLOC_SCRATCH_BYTES];

size_t tconv_forward_noalloc_max_scratch(void) { return TCONV_NOALLOC_SCRATCH_BYTES; }

int tconv_forward_noalloc(const tconv_desc_t* desc, const void* x, const void* w, const void* w2,
                          const float* alpha, const float* beta, const float* bias, void* y,
                          void* winners, void* stream) {
    Geo g;
    int rc = make_geo(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (!x || !w || !y) return TCONV_ERR_INVALID_ARG;
    if (g.mode == TCONV_PARALLEL && !w2) return TCONV_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(w) || misaligned(w2) || misaligned(alpha) || misaligned(beta) ||
        misaligned(bias) || misaligned(y) || misaligned(winners))
        return TCONV_ERR_MISALIGNED;
    const size_t need = tconv_workspace_bytes(desc, 0);
    if (need > TCONV_NOALLOC_SCRATCH_BYTES) {
        snprintf(g_last_error, sizeof(g_last_error),
                 "layer needs %zu bytes of scratch, the built-in scratch holds %u", need,
                 (unsigned)TCONV_NOALLOC_SCRATCH_BYTES);
        return TCONV_ERR_TOO_LARGE;
    }
    // In host code the array's name is only a stand-in; the device address comes from the
    // runtime, once per device, with that device current.
    static void* scratch_ptr[64] = {nullptr};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return TCONV_ERR_UNSUPPORTED;
    if (!scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
        if (e != cudaSuccess) return cuda_fail(e);
        scratch_ptr[dev] = p;
    }
    if (!two_branch(g.mode)) { alpha = nullptr; beta = nullptr; }
    cudaStream_t st = (cudaStream_t)stream;
    g_last_error[0] = 0;
    if (desc->dtype == TCONV_F32)
        return forward_t<float>(g, x, w, w2, alpha, beta, bias, y, winners, scratch_ptr[dev],
                                TCONV_NOALLOC_SCRATCH_BYTES, st);
    return forward_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, bias, y, winners, scratch_ptr[dev],
                                    TCONV_NOALLOC_SCRATCH_BYTES, st);
}

const char* tconv_last_error(void) { return g_last_error; }
const char* tconv_last_kernel(void) { return g_last_kernel; }
long long tconv_launch_count(void) { return g_launches; }

}  // extern "C"

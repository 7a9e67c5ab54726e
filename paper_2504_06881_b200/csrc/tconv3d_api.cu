// C ABI of the three-dimensional layers: host-side checks, launch plans, kernel launches.
#include <cstdio>

#include "tconv3d.h"
#include "tconv_3d.cuh"

namespace tconv {
namespace {

thread_local long long g3_launches = 0;

int extent(int in, int pad, int dil, int k, int stride) {
    const long span = (long)in + 2L * pad - (long)dil * (k - 1) - 1;
    return span < 0 ? 0 : (int)(span / stride) + 1;
}

int make_geo3(const tconv3d_desc_t* d, Geo3* g) {
    if (!d) return TCONV_ERR_INVALID_ARG;
    if (d->N <= 0 || d->C <= 0 || d->D <= 0 || d->H <= 0 || d->W <= 0 || d->K <= 0 || d->T <= 0 ||
        d->R <= 0 || d->S <= 0)
        return TCONV_ERR_INVALID_ARG;
    if (d->stride_d <= 0 || d->stride_h <= 0 || d->stride_w <= 0 || d->dil_d <= 0 || d->dil_h <= 0 ||
        d->dil_w <= 0 || d->pad_d < 0 || d->pad_h < 0 || d->pad_w < 0)
        return TCONV_ERR_INVALID_ARG;
    if (d->mode < TCONV_MAX_PLUS || d->mode > TCONV_PARALLEL) return TCONV_ERR_INVALID_ARG;
    if (d->chan < TCONV_CHAN_DEFAULT || d->chan > TCONV_CHAN_MIN) return TCONV_ERR_INVALID_ARG;
    if (d->dtype != TCONV_F32 && d->dtype != TCONV_BF16) return TCONV_ERR_INVALID_ARG;
    const bool two = two_branch(d->mode);
    int chan = d->chan;
    if (chan == TCONV_CHAN_DEFAULT)
        chan = two ? TCONV_CHAN_SUM : (d->mode == TCONV_MAX_PLUS ? TCONV_CHAN_MAX : TCONV_CHAN_MIN);
    if (two && chan != TCONV_CHAN_SUM) return TCONV_ERR_UNSUPPORTED;
    if ((long)d->T * d->R * d->S > 256) return TCONV_ERR_UNSUPPORTED;
    g->N = d->N; g->C = d->C; g->D = d->D; g->H = d->H; g->W = d->W; g->K = d->K;
    g->T = d->T; g->R = d->R; g->S = d->S;
    g->sd = d->stride_d; g->sh = d->stride_h; g->sw = d->stride_w;
    g->pd = d->pad_d; g->ph = d->pad_h; g->pw = d->pad_w;
    g->dd = d->dil_d; g->dh = d->dil_h; g->dw = d->dil_w;
    g->OD = extent(d->D, d->pad_d, d->dil_d, d->T, d->stride_d);
    g->OH = extent(d->H, d->pad_h, d->dil_h, d->R, d->stride_h);
    g->OW = extent(d->W, d->pad_w, d->dil_w, d->S, d->stride_w);
    if (g->OD <= 0 || g->OH <= 0 || g->OW <= 0) return TCONV_ERR_INVALID_ARG;
    g->taps = d->T * d->R * d->S;
    const double lim = 2147483647.0;
    const double vol = (double)g->OD * g->OH * g->OW;
    if ((double)d->N * d->C * d->D * d->H * d->W > lim || (double)d->N * d->K * vol * d->C > lim ||
        (double)d->K * d->C * g->taps > lim || (double)d->N * d->K * vol > lim)
        return TCONV_ERR_TOO_LARGE;
    g->vol = (int)vol;
    g->mode = d->mode;
    g->chan = chan == TCONV_CHAN_SUM ? CH_SUM : (chan == TCONV_CHAN_MAX ? CH_MAX : CH_MIN);
    return TCONV_OK;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

size_t winner_bytes3(const Geo3& g) {
    if (g.chan == CH_SUM) return (size_t)g.N * g.K * g.C * g.vol * sizeof(uint16_t);
    return (size_t)g.N * g.K * g.vol * sizeof(int32_t);
}

// Splits of the (n, position) range for the grad_w partial sums: enough blocks to fill the SMs
// when K*C is small, each split at least four stages long.
int gw_splits(const Geo3& g) {
    const long long total = (long long)g.N * g.vol;
    long long want = (2 * 148 + (long long)g.K * g.C - 1) / ((long long)g.K * g.C);
    const long long most = (total + 4 * kGw3Stage - 1) / (4 * kGw3Stage);
    if (want > most) want = most;
    if (want < 1) want = 1;
    if (want > 64) want = 64;
    return (int)want;
}

// Splits of the same range for the grad_bias partial sums (K blocks otherwise).
int bias_splits(const Geo3& g) {
    const long long total = (long long)g.N * g.vol;
    long long want = (2 * 148 + g.K - 1) / g.K;
    const long long most = (total + 4095) / 4096;
    if (want > most) want = most;
    if (want < 1) want = 1;
    if (want > 64) want = 64;
    return (int)want;
}

size_t backward_scratch_floats(const Geo3& g) {
    const size_t ns = (size_t)gw_splits(g);
    return 2 * ns * g.K * g.C * g.taps + 2 * ns * g.K * g.C + (size_t)bias_splits(g) * g.K;
}

int check(cudaError_t e) { return e == cudaSuccess ? TCONV_OK : TCONV_ERR_CUDA; }

template <typename T>
int forward3_t(const Geo3& g, const void* x, const void* w, const void* w2, const float* alpha,
               const float* beta, const float* bias, void* y, void* winners, cudaStream_t st) {
    const bool par = g.mode == TCONV_PARALLEL;
    // two output channels per thread when K is small and not a multiple of four, else four
    const int kt = (g.K % 4 == 0 || g.K > 8) ? 4 : 2;
    const size_t per_c = (size_t)g.taps * kt * sizeof(T) * (par ? 2 : 1);
    int cch = (int)(48 * 1024 / per_c);
    if (cch < 1) cch = 1;
    if (cch > g.C) cch = g.C;
    const size_t smem = per_c * cch;
    const long long flat = (long long)g.N * g.vol;
    const dim3 grid((unsigned)((flat + kFwd3Threads - 1) / kFwd3Threads), (unsigned)((g.K + kt - 1) / kt));
#define TCONV3_LAUNCH(KTV, WINV, SCV)                                                                     \
    fwd3d_kernel<T, KTV, WINV, SCV><<<grid, kFwd3Threads, smem, st>>>(                                     \
        g, cch, (const T*)x, (const T*)w, (const T*)w2, alpha, beta, bias, (T*)y, winners)
#define TCONV3_BY_S(KTV, WINV)                                   \
    {                                                            \
        if (g.S == 3) TCONV3_LAUNCH(KTV, WINV, 3);               \
        else if (g.S == 5) TCONV3_LAUNCH(KTV, WINV, 5);          \
        else TCONV3_LAUNCH(KTV, WINV, 0);                        \
    }
    if (kt == 4) {
        if (winners) TCONV3_BY_S(4, true) else TCONV3_BY_S(4, false)
    } else {
        if (winners) TCONV3_BY_S(2, true) else TCONV3_BY_S(2, false)
    }
#undef TCONV3_BY_S
#undef TCONV3_LAUNCH
    g3_launches += 1;
    return check(cudaGetLastError());
}

template <typename T>
int backward3_t(const Geo3& g, const void* x, const void* w, const void* w2, const float* alpha,
                const float* beta, const void* gy, const void* winners, void* gx, float* gw, float* gw2,
                float* galpha, float* gbeta, float* gbias, char* ws, cudaStream_t st) {
    const bool two = two_branch(g.mode);
    if (gx) {
        const size_t total = (size_t)g.N * g.C * g.D * g.H * g.W;
        // channel slices only while the input has too few elements to fill the GPU with one thread
        // each: every slice repeats the tap geometry of its element
        const size_t want = ((size_t)148 * 2048 + total - 1) / total;
        int slices = 1;
        while (slices < kGx3Slices && (size_t)slices < want && 2 * slices <= g.K) slices *= 2;
        const unsigned per_block = 32u * kGx3Slices / slices;
        bwd3d_gx_kernel<T><<<(unsigned)((total + per_block - 1) / per_block), dim3(per_block, (unsigned)slices), 0, st>>>(
            g, alpha, beta, (const T*)gy, winners, (T*)gx);
        g3_launches += 1;
    }
    const int nsplit = gw_splits(g);
    const size_t count = (size_t)g.K * g.C * g.taps;
    float* pmin = (float*)ws;
    float* pmax = pmin + (size_t)nsplit * count;
    float* pab = pmax + (size_t)nsplit * count;          // [nsplit][K*C][2]
    float* pbias = pab + (size_t)nsplit * g.K * g.C * 2;  // [bias splits][K]
    if (gw || gw2) {
        bwd3d_gw_kernel<T><<<dim3((unsigned)(g.K * g.C), (unsigned)nsplit), 256, 0, st>>>(
            g, nsplit, (const T*)gy, winners, pmin, pmax);
        bwd3d_gw_finish_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(g, nsplit, alpha, beta, pmin,
                                                                               pmax, gw, gw2);
        g3_launches += 2;
    }
    if (two && (galpha || gbeta)) {
        bwd3d_gab_kernel<T><<<dim3((unsigned)(g.K * g.C), (unsigned)nsplit), 256, 0, st>>>(
            g, nsplit, (const T*)x, (const T*)w, (const T*)w2, (const T*)gy, winners, pab);
        const int kc = g.K * g.C;
        if (galpha) bwd3d_sum_splits_kernel<<<(kc + 255) / 256, 256, 0, st>>>(kc, nsplit, 2, 0, pab, galpha);
        if (gbeta) bwd3d_sum_splits_kernel<<<(kc + 255) / 256, 256, 0, st>>>(kc, nsplit, 2, 1, pab, gbeta);
        g3_launches += 1 + (galpha ? 1 : 0) + (gbeta ? 1 : 0);
    }
    if (gbias) {
        const int bs = bias_splits(g);
        bwd3d_bias_kernel<T><<<dim3((unsigned)g.K, (unsigned)bs), 256, 0, st>>>(g, bs, (const T*)gy, pbias);
        bwd3d_sum_splits_kernel<<<(g.K + 255) / 256, 256, 0, st>>>(g.K, bs, 1, 0, pbias, gbias);
        g3_launches += 2;
    }
    return check(cudaGetLastError());
}

bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

}  // namespace
}  // namespace tconv

using namespace tconv;

extern "C" {

int tconv3d_output_shape(const tconv3d_desc_t* desc, int32_t* OD, int32_t* OH, int32_t* OW) {
    Geo3 g;
    const int rc = make_geo3(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (OD) *OD = g.OD;
    if (OH) *OH = g.OH;
    if (OW) *OW = g.OW;
    return TCONV_OK;
}

size_t tconv3d_winner_bytes(const tconv3d_desc_t* desc) {
    Geo3 g;
    if (make_geo3(desc, &g) != TCONV_OK) return 0;
    return winner_bytes3(g);
}

size_t tconv3d_workspace_bytes(const tconv3d_desc_t* desc, int backward) {
    Geo3 g;
    if (make_geo3(desc, &g) != TCONV_OK || !backward) return 0;
    return align_up(winner_bytes3(g), 256) + backward_scratch_floats(g) * sizeof(float) + 256;
}

int tconv3d_forward(const tconv3d_desc_t* desc, const void* x, const void* w, const void* w2,
                    const float* alpha, const float* beta, const float* bias, void* y, void* winners,
                    void* stream) {
    Geo3 g;
    const int rc = make_geo3(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (!x || !w || (!y && !winners)) return TCONV_ERR_INVALID_ARG;
    if (g.mode == TCONV_PARALLEL && !w2) return TCONV_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(y) || misaligned(winners)) return TCONV_ERR_MISALIGNED;
    if (!two_branch(g.mode)) alpha = beta = nullptr;
    cudaStream_t st = (cudaStream_t)stream;
    return desc->dtype == TCONV_F32 ? forward3_t<float>(g, x, w, w2, alpha, beta, bias, y, winners, st)
                                    : forward3_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, bias, y, winners, st);
}

int tconv3d_backward(const tconv3d_desc_t* desc, const void* x, const void* w, const void* w2,
                     const float* alpha, const float* beta, const void* grad_y, const void* winners,
                     void* grad_x, float* grad_w, float* grad_w2, float* grad_alpha, float* grad_beta,
                     float* grad_bias, void* workspace, size_t workspace_bytes, void* stream) {
    Geo3 g;
    int rc = make_geo3(desc, &g);
    if (rc != TCONV_OK) return rc;
    if (!x || !w || !grad_y) return TCONV_ERR_INVALID_ARG;
    if (g.mode == TCONV_PARALLEL && !w2) return TCONV_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(grad_y) || misaligned(winners) || misaligned(grad_x) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return TCONV_ERR_MISALIGNED;
    if (!workspace || workspace_bytes < tconv3d_workspace_bytes(desc, 1)) return TCONV_ERR_WORKSPACE_TOO_SMALL;
    if (!two_branch(g.mode)) alpha = beta = nullptr;
    if (g.mode != TCONV_PARALLEL) grad_w2 = nullptr;
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = (char*)workspace;
    const bool f32 = desc->dtype == TCONV_F32;
    if (!winners) {
        rc = f32 ? forward3_t<float>(g, x, w, w2, alpha, beta, nullptr, nullptr, ws, st)
                 : forward3_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, nullptr, nullptr, ws, st);
        if (rc != TCONV_OK) return rc;
        winners = ws;
    }
    ws += align_up(winner_bytes3(g), 256);
    return f32 ? backward3_t<float>(g, x, w, w2, alpha, beta, grad_y, winners, grad_x, grad_w, grad_w2,
                                    grad_alpha, grad_beta, grad_bias, ws, st)
               : backward3_t<__nv_bfloat16>(g, x, w, w2, alpha, beta, grad_y, winners, grad_x, grad_w, grad_w2,
                                            grad_alpha, grad_beta, grad_bias, ws, st);
}

long long tconv3d_launch_count(void) { return g3_launches; }

}  // extern "C"

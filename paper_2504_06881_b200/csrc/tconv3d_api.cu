// C ABI of the three-dimensional layers: host-side checks, launch plans, kernel launches.
#include <cstdio>

#include <cstdlib>

#include "tconv3d.h"
#include "tconv_1d.cuh"
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

// TCONV_FORCE_GENERIC=1 keeps every call on the any-shape kernels (read once per process).
bool force_generic3() {
    static const int v = [] {
        const char* e = getenv("TCONV_FORCE_GENERIC");
        return (e && e[0] == '1') ? 1 : 0;
    }();
    return v != 0;
}

// One-dimensional layers (unit depth and height, 1 x 1 x S window) with windows of four taps or
// more at stride 1, 2 or 4 run on the kernels of tconv_1d.cuh.
bool is_1d(const Geo3& g) {
    return g.D == 1 && g.H == 1 && g.T == 1 && g.R == 1 && g.pd == 0 && g.ph == 0 && g.dw == 1 &&
           (g.sw == 1 || g.sw == 2 || g.sw == 4) && g.S >= 4 && g.N <= 65535 && !force_generic3();
}

constexpr size_t kSmem1d = 96 * 1024;  // most dynamic shared memory a backward 1-D block asks for

// Launch plan of the 1-D backward kernels.  ok = 0: the layer stays on the any-shape kernels (a
// Max / Min channel combine over several channels, whose winners name one channel per output).
struct Plan1 {
    int ok;
    int pt, tb, span, tiles, ks;  // grad_x: positions per thread, threads, array length, tiles, channel slices
    int ptb, nsplit;              // parameter gradients: threads, splits of the (n, position) range
    size_t gx_smem, p_smem, part_floats, scratch_floats;
};

Plan1 plan_1d(const Geo3& g) {
    Plan1 p = {};
    if (!is_1d(g) || !(g.chan == CH_SUM || g.C == 1)) return p;
    const int st = g.sw, S = g.S, OL = g.OW;
    p.pt = (S + st - 1) / st - 1;
    if (p.pt < 8) p.pt = 8;
    p.tb = kGx1Threads;
    for (;;) {
        p.span = p.tb * p.pt * st - st + S;
        p.gx_smem = 2 * (size_t)p.span * sizeof(float);
        if (p.gx_smem <= kSmem1d || p.tb == 32) break;
        p.tb /= 2;
    }
    if (p.gx_smem > kSmem1d) return p;
    p.tiles = (OL + p.tb * p.pt - 1) / (p.tb * p.pt);
    const long long blocks = (long long)p.tiles * g.C * g.N;
    long long ks = (4 * 148 + blocks - 1) / blocks;
    if (ks > 8) ks = 8;
    if (ks > g.K) ks = g.K;
    if ((long long)g.C * ks > 65535) return p;
    p.ks = (int)ks;
    p.part_floats = (size_t)p.ks * g.N * g.C * p.tiles * p.span;
    const int branches = two_branch(g.mode) ? 2 : 1;
    // threads per block: 128, or fewer while the private columns of a block exceed 48 KB (two
    // branches of a long window), so that several blocks stay resident per SM
    p.ptb = 128;
    for (;;) {
        p.p_smem = ((size_t)branches * (S + 1) * p.ptb + 2 * S + p.ptb) * sizeof(float);
        if (p.p_smem <= 48 * 1024 || p.ptb == 32) break;
        p.ptb /= 2;
    }
    if (p.p_smem > kSmem1d) return p;
    // splits of the (n, position) range: as many blocks as are resident at once (one round), each
    // split at least 2048 items long
    const long long kc = (long long)g.K * g.C, total = (long long)g.N * OL;
    long long per_sm = (long long)(200 * 1024 / (p.p_smem + 1024));
    if (per_sm > 384 / p.ptb) per_sm = 384 / p.ptb;   // registers: the kernel's launch bounds
    long long want = 148 * per_sm / kc;
    const long long most = (total + 2047) / 2048;
    if (want > most) want = most;
    if (want < 1) want = 1;
    if (want > 64) want = 64;
    p.nsplit = (int)want;
    p.scratch_floats = 2 * (size_t)p.nsplit * kc * S + 2 * (size_t)p.nsplit * kc + (size_t)p.nsplit * g.K +
                       p.part_floats;
    p.ok = 1;
    return p;
}

size_t backward_scratch_floats(const Geo3& g) {
    const size_t ns = (size_t)gw_splits(g);
    const size_t generic = 2 * ns * g.K * g.C * g.taps + 2 * ns * g.K * g.C + (size_t)bias_splits(g) * g.K;
    const Plan1 p = plan_1d(g);
    return (p.ok && p.scratch_floats > generic) ? p.scratch_floats : generic;
}

int check(cudaError_t e) { return e == cudaSuccess ? TCONV_OK : TCONV_ERR_CUDA; }

template <typename T>
int forward1d_t(const Geo3& g, const void* x, const void* w, const void* w2, const float* alpha,
                const float* beta, const float* bias, void* y, void* winners, cudaStream_t st) {
    const int q4 = (((g.S + g.sw - 1) / g.sw) + 3) & ~3;
    const int br = g.mode == TCONV_MIN_PLUS ? 0 : (g.mode == TCONV_MAX_PLUS ? 1 : (g.mode == TCONV_COMPOUND ? 2 : 3));
    const int kb = 4 * f1_kt(br, winners != nullptr);
    // signal segment, weights by tap, and with winners a second copy of the weights by channel
    // (a bf16 layer stages its weights by tap as 4-byte {w, w} pairs; with winners a second copy by
    // channel follows in the layer's type)
    const size_t wcopy = (size_t)q4 * g.sw * kb * (br == 3 ? 2 : 1);
    const size_t smem = (size_t)g.sw * f1_xw(q4) * sizeof(T) + wcopy * 4 + (winners ? wcopy * sizeof(T) : 0);
    const dim3 grid((unsigned)((g.OW + kF1Pos - 1) / kF1Pos), (unsigned)((g.K + kb - 1) / kb), (unsigned)g.N);
    // (long windows with winners in parallel mode stage up to 67 KB: above the default limit)
#define TCONV1_LAUNCH(STV, BRV, WINV)                                                     \
    {                                                                                     \
        if (smem > 48 * 1024 &&                                                           \
            cudaFuncSetAttribute(fwd1d_kernel<T, STV, BRV, WINV>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                 (int)kSmem1d) != cudaSuccess)                            \
            return TCONV_ERR_CUDA;                                                        \
        fwd1d_kernel<T, STV, BRV, WINV><<<grid, kF1Threads, smem, st>>>(                   \
            g, q4, (const T*)x, (const T*)w, (const T*)w2, alpha, beta, bias, (T*)y, winners); \
    }
#define TCONV1_BY_WIN(STV, BRV)                                  \
    {                                                            \
        if (winners) TCONV1_LAUNCH(STV, BRV, true)               \
        else TCONV1_LAUNCH(STV, BRV, false)                      \
    }
#define TCONV1_BY_BR(STV)                                        \
    {                                                            \
        if (br == 0) TCONV1_BY_WIN(STV, 0)                       \
        else if (br == 1) TCONV1_BY_WIN(STV, 1)                  \
        else if (br == 2) TCONV1_BY_WIN(STV, 2)                  \
        else TCONV1_BY_WIN(STV, 3)                               \
    }
    if (g.sw == 1) TCONV1_BY_BR(1)
    else if (g.sw == 2) TCONV1_BY_BR(2)
    else TCONV1_BY_BR(4)
#undef TCONV1_BY_BR
#undef TCONV1_BY_WIN
#undef TCONV1_LAUNCH
    g3_launches += 1;
    return check(cudaGetLastError());
}

template <typename T>
int forward3_t(const Geo3& g, const void* x, const void* w, const void* w2, const float* alpha,
               const float* beta, const float* bias, void* y, void* winners, cudaStream_t st) {
    if (is_1d(g)) return forward1d_t<T>(g, x, w, w2, alpha, beta, bias, y, winners, st);
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

// Backward of a 1-D layer on the kernels of tconv_1d.cuh.  Scratch: part_min, part_max
// [nsplit][K*C][S], part_ab [nsplit][K*C][2], part_bias [nsplit][K], then the grad_x partial sums.
template <typename T>
int backward1d_t(const Geo3& g, const Plan1& p, const void* x, const void* w, const void* w2,
                 const float* alpha, const float* beta, const void* gy, const void* winners, void* gx,
                 float* gw, float* gw2, float* galpha, float* gbeta, float* gbias, char* ws, cudaStream_t st) {
    static const cudaError_t attr = [] {
        cudaError_t e = cudaFuncSetAttribute(bwd1d_gx_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem1d);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(bwd1d_params_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem1d);
        return e;
    }();
    if (attr != cudaSuccess) return TCONV_ERR_CUDA;
    const size_t kc = (size_t)g.K * g.C, count = kc * g.S;
    float* pmin = (float*)ws;
    float* pmax = pmin + (size_t)p.nsplit * count;
    float* pab = pmax + (size_t)p.nsplit * count;
    float* pbias = pab + (size_t)p.nsplit * kc * 2;
    float* part = pbias + (size_t)p.nsplit * g.K;
    if (gx) {
        bwd1d_gx_kernel<T><<<dim3((unsigned)p.tiles, (unsigned)(g.C * p.ks), (unsigned)g.N), p.tb, p.gx_smem, st>>>(
            g, p.pt, p.ks, p.span, alpha, beta, (const T*)gy, winners, part);
        const size_t total = (size_t)g.N * g.C * g.W;
        bwd1d_gx_finish_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
            g, p.tiles, p.ks, p.span, p.tb * p.pt * g.sw, part, (T*)gx);
        g3_launches += 2;
    }
    const bool two = two_branch(g.mode);
    if (gw || gw2 || gbias || (two && (galpha || gbeta))) {
        bwd1d_params_kernel<T><<<dim3((unsigned)kc, (unsigned)p.nsplit), p.ptb, p.p_smem, st>>>(
            g, p.nsplit, (const T*)x, (const T*)w, (const T*)w2, (const T*)gy, winners, pmin, pmax, pab, pbias);
        g3_launches += 1;
        if (gw || gw2) {
            bwd3d_gw_finish_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(g, p.nsplit, alpha, beta, pmin,
                                                                                   pmax, gw, gw2);
            g3_launches += 1;
        }
        if (two && galpha) {
            bwd3d_sum_splits_kernel<<<(unsigned)((kc + 255) / 256), 256, 0, st>>>((int)kc, p.nsplit, 2, 0, pab, galpha);
            g3_launches += 1;
        }
        if (two && gbeta) {
            bwd3d_sum_splits_kernel<<<(unsigned)((kc + 255) / 256), 256, 0, st>>>((int)kc, p.nsplit, 2, 1, pab, gbeta);
            g3_launches += 1;
        }
        if (gbias) {
            bwd3d_sum_splits_kernel<<<(g.K + 255) / 256, 256, 0, st>>>(g.K, p.nsplit, 1, 0, pbias, gbias);
            g3_launches += 1;
        }
    }
    return check(cudaGetLastError());
}

template <typename T>
int backward3_t(const Geo3& g, const void* x, const void* w, const void* w2, const float* alpha,
                const float* beta, const void* gy, const void* winners, void* gx, float* gw, float* gw2,
                float* galpha, float* gbeta, float* gbias, char* ws, cudaStream_t st) {
    {
        const Plan1 p1 = plan_1d(g);
        if (p1.ok)
            return backward1d_t<T>(g, p1, x, w, w2, alpha, beta, gy, winners, gx, gw, gw2, galpha, gbeta, gbias, ws, st);
    }
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

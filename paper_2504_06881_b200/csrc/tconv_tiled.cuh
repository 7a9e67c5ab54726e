// Tiled forward kernels (fp32).
//
// A CTA owns TILE_K output channels x one tile of output pixels and walks the
// input channels in chunks of CC.  Per chunk the input halo tile (zero padding
// comes from the copy engine's out-of-bounds fill) and the repacked weights of
// the chunk are brought into shared memory by TMA: one tiled tensor copy for x,
// one bulk copy for each weight / alpha / beta block, all signalling one mbarrier
// per stage (two stages).  Feature maps whose rows are not 16-byte multiples, or
// tiles that span several images of a small map, take per-element asynchronous
// copies instead.  Every thread keeps 8 output channels x Q x 4 pixels in
// registers and folds taps with packed adds (two channels per instruction) and
// 3-input min / max.
#pragma once
#include <cuda.h>

#include <cstdlib>
#include <cstring>

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
// Extremum of v[0..RS)[h] with 3-input min / max: a fresh chain opens with three values,
// every later step folds two more.
template <int RS>
__device__ __forceinline__ float fold_taps(const float (*v)[2], int h, bool is_min) {
    float m;
    if constexpr (RS >= 3) m = ext3(v[0][h], v[1][h], v[2][h], is_min);
    else if constexpr (RS == 2) m = ext2(v[0][h], v[1][h], is_min);
    else m = v[0][h];
#pragma unroll
    for (int i = 3; i + 1 < RS; i += 2) m = ext3(m, v[i][h], v[i + 1][h], is_min);
    if constexpr (RS > 3 && ((RS - 3) & 1)) m = ext2(m, v[RS - 1][h], is_min);
    return m;
}
// {c0, c1} = a * {v0, v1} + {c0, c1}: one packed fused multiply-add (scalar a splat)
__device__ __forceinline__ void fma2s(float a, float v0, float v1, float& c0, float& c1) {
    unsigned long long aa, vv, cc;
    asm("mov.b64 %0, {%1, %1};" : "=l"(aa) : "f"(a));
    asm("mov.b64 %0, {%1, %2};" : "=l"(vv) : "f"(v0), "f"(v1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(cc) : "f"(c0), "f"(c1));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(cc) : "l"(aa), "l"(vv));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(c0), "=f"(c1) : "l"(cc));
}
__device__ __forceinline__ unsigned smem_u32(const void* p) {
    return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async4(void* smem, const void* gmem, bool valid) {
    const int n = valid ? 4 : 0;  // 0 source bytes: the destination is zero-filled
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(smem)), "l"(gmem), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// mbarrier + TMA (single-CTA use: every copy lands in the shared memory of the CTA that issued it)
__device__ __forceinline__ void mbar_init(void* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait: gives up after kPollLimit polls and reports failure.  A poll that finds the phase
// incomplete blocks for a hardware time slice (measured: 4 us), so 2^16 polls bound a wait at a
// quarter of a second, five orders of magnitude above the microseconds a copy takes.  (The limit is
// a compile-time constant on purpose: a run-time limit costs the main loops a register.)
constexpr int kPollLimit = 1 << 16;
__device__ __forceinline__ bool mbar_wait(void* bar, unsigned parity) {
    const unsigned addr = smem_u32(bar);
    for (int i = 0; i < kPollLimit; ++i) {
        unsigned ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_3d(void* smem, const CUtensorMap* map, int c0, int c1,
                                            int c2, void* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(smem)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_load(void* smem, const void* gmem, unsigned bytes, void* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(smem)), "l"(gmem), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// L floats starting SHIFT floats past a 16-byte aligned shared-memory address, with the
// widest aligned vector loads the position allows.
template <int SHIFT, int L, int I = 0>
__device__ __forceinline__ void load_segment(const float* base, float* out) {
    if constexpr (I < L) {
        constexpr int pos = SHIFT + I;
        if constexpr ((pos % 4 == 0) && (I + 4 <= L)) {
            const float4 v = *reinterpret_cast<const float4*>(base + pos);
            out[I] = v.x; out[I + 1] = v.y; out[I + 2] = v.z; out[I + 3] = v.w;
            load_segment<SHIFT, L, I + 4>(base, out);
        } else if constexpr ((pos % 2 == 0) && (I + 2 <= L)) {
            const float2 v = *reinterpret_cast<const float2*>(base + pos);
            out[I] = v.x; out[I + 1] = v.y;
            load_segment<SHIFT, L, I + 2>(base, out);
        } else {
            out[I] = base[pos];
            load_segment<SHIFT, L, I + 1>(base, out);
        }
    }
}
template <int N>
__device__ __forceinline__ void loadn(const float* p, float* out) {
    static_assert(N == 2 || N % 4 == 0, "vector loads");
    if constexpr (N == 2) {
        const float2 a = *reinterpret_cast<const float2*>(p);
        out[0] = a.x; out[1] = a.y;
    } else {
#pragma unroll
        for (int i = 0; i < N; i += 4) {
            const float4 a = *reinterpret_cast<const float4*>(p + i);
            out[i] = a.x; out[i + 1] = a.y; out[i + 2] = a.z; out[i + 3] = a.w;
        }
    }
}
__device__ __forceinline__ void load8(const float* p, float* out) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    const float4 b = *reinterpret_cast<const float4*>(p + 4);
    out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
    out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
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
    const void* w;     // weights as the caller passed them ([K][C][R][S])
    const float* wt;   // repacked weights (min branch / the only weights)
    const float* wt2;  // repacked max-branch weights (parallel)
    const float* at;   // repacked alpha, beta
    const float* bt;
    const float* bias;
    void* y;
    void* winners;
    int* status;       // device status word: set non-zero when a bounded wait gives up
    int TW, QPR, TH;   // tile: output columns, quads per row, output rows
    int n_col_tiles, n_row_tiles;
    int tiles_per_img; // > 0: row tiles stay inside one image; 0: rows run over the flattened (n, oh) space
    int total_rows;    // N * OH
    int ragged;        // 1: a tile is NQ consecutive quads of the flattened (n, oh, quad) space (rows whose
                       //    quads do not divide the lanes of a warp), 0: a tile is TH whole rows
    int total_quads;   // N * OH * QPR
    int xbox;          // elements of one staged x block (channels x rows x pitch)
    int xblock;        // ragged TMA tiles: elements between the staged blocks of the tile's two images
                       // (xbox rounded up so that the second block starts on a 128-byte boundary)
    int NSLOTS, XW, XP;  // staged input rows per tile, staged columns, row pitch (floats)
    int GAP;           // extra input-row slots between two images of one tile (flattened tiles)
    int CC, Cpad, nchunks;
    int stage_floats, x_stage, w_stage, ab_stage;  // shared-memory layout of one stage (4-byte words)
    // (later additions stay at the end: the register allocation of the kernels that sit at their
    // register cap proved sensitive to the offsets of the fields above)
    int stats_k;       // channel pitch of the statistics partials (K rounded up to the k tile)
    int debug_drop;    // failure-test switch: the copies of the first chunk are never issued
    float* stats;      // NULL, or per-tile partial sums {sum y, sum y^2} per output channel: [tile][stats_k][2]
};

// Column shift of the TMA path: the tile's first input column ow0*SW - pw is rounded
// down to a multiple of 4 floats so that the copy starts on a 16-byte boundary.  The
// TMA path is used with "same" padding pw = (S-1)*DW/2 only, which fixes the shift.
template <int S, int DW, int ESIZE = 4> struct TmaShift {
    static constexpr int unit = 16 / ESIZE;  // elements per 16 bytes
    static constexpr int value = (unit - (((S - 1) * DW / 2) % unit)) % unit;
};

// MODE: tconv_mode_t, CHAN: CH_SUM / CH_MAX / CH_MIN, WIN: emit winners, XTMA: x tile by TMA.
// Q quads of 4 pixels per thread, KG groups of 8 output channels and PW pixel warps per CTA.
// Resident CTAs per SM the register allocation aims at: the winner-free kernels are bound by
// the ALU / FMA pipes and want four or more warps per scheduler to hide their latencies.
constexpr int kMinBlocksSingle = 4;   // single-branch kernels
constexpr int kMinBlocksWinSum = 3;   // Sum forms that emit winners (168 registers)
constexpr int kQuadsCarried = 2;      // quads per thread of the carried max-plus / min-plus chain
// STATS (winner-emitting kernels only): also leave the per-tile channel statistics.
template <int MODE, int CHAN, bool WIN, bool XTMA, bool RAG, int R, int S, int SW, int DW, int Q, int KG, int PW, int TK, bool STATS = false>
__global__ void __launch_bounds__(KG * PW * 32,
                                  (WIN && CHAN == CH_SUM) ? kMinBlocksWinSum
                                  : WIN ? 1
                                  : (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL) ? (TK == 4 ? 4 : 1)
                                  : kMinBlocksSingle)
fwd_tiled_f32_kernel(const __grid_constant__ CUtensorMap xmap, const TiledParams p) {
    static_assert(TK == 2 || TK == 4 || TK == 8, "output channels per thread");
    constexpr int RS = R * S;
    constexpr int TILE_K = KG * TK;
    constexpr int NT = KG * PW * 32;
    constexpr int NWARPS = KG * PW;
    constexpr int L = 3 * SW + (S - 1) * DW + 1;  // input columns one quad touches per row
    constexpr int SHIFT = XTMA ? TmaShift<S, DW>::value : 0;
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool PAR = (MODE == TCONV_PARALLEL);
    constexpr bool TAP_MIN = (MODE == TCONV_MIN_PLUS);  // tap-level extremum of single-branch modes
    // running extremum carried across channels when tap and channel level agree
    constexpr bool CARRIED = !TWO && !WIN &&
                             ((MODE == TCONV_MAX_PLUS && CHAN == CH_MAX) ||
                              (MODE == TCONV_MIN_PLUS && CHAN == CH_MIN));
    const Geo& g = p.g;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* stage0 = reinterpret_cast<float*>(smem_raw);
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(stage0 + 2 * p.stage_floats);
    int* slot_off = reinterpret_cast<int*>(bars + 2);

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
        // input-row slot table: element offset of the row start inside x (channel 0), or -1
        for (int sl = tid; sl < p.NSLOTS; sl += NT) slot_off[sl] = -1;
        __syncthreads();
        const int span = (R - 1) * g.dh + 1;
        for (int e = tid; e < rows_here * span; e += NT) {
            const int lr = e / span, dr = e - lr * span;
            const int gr = row0 + lr;
            const int n = gr / g.OH, oh = gr - n * g.OH;
            const int ih = oh * g.sh - g.ph + dr;
            const int sl = lr * g.sh + (n - n0) * p.GAP + dr;
            if (ih >= 0 && ih < g.H) slot_off[sl] = (n * g.C * g.H + ih) * g.W;  // writers agree
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
            xoff[q] = (n == n0 ? lr * g.sh * p.XP : p.xblock + (gr - (n0 + 1) * g.OH) * g.sh * p.XP) + qx * 4 * SW;
        else
            xoff[q] = (lr * g.sh + (n - n0) * p.GAP) * p.XP + qx * 4 * SW;
    }

    const float* xg = reinterpret_cast<const float*>(p.x);
    const size_t chw = (size_t)g.H * g.W;
    const float* wt_k = p.wt + (size_t)kt * p.Cpad * RS * TILE_K;
    const float* wt2_k = PAR ? p.wt2 + (size_t)kt * p.Cpad * RS * TILE_K : nullptr;
    const float* at_k = TWO ? p.at + (size_t)kt * p.Cpad * TILE_K : nullptr;
    const float* bt_k = TWO ? p.bt + (size_t)kt * p.Cpad * TILE_K : nullptr;
    const int w_off = p.x_stage, w2_off = p.x_stage + p.w_stage;
    const int a_off = p.x_stage + p.w_stage * (PAR ? 2 : 1), b_off = a_off + p.ab_stage;

    auto issue_chunk = [&](int ch, int s) {
        float* st = stage0 + s * p.stage_floats;
        const int c0 = ch * p.CC;
        if constexpr (XTMA) {
            if (tid == 0 && !(p.debug_drop && ch == 0)) {
                const unsigned bytes = (unsigned)((p.xbox * (two_imgs ? 2 : 1) + p.w_stage * (PAR ? 2 : 1) + 2 * p.ab_stage) * sizeof(float));
                mbar_expect_tx(&bars[s], bytes);
                tma_load_3d(st, &xmap, iw0 - SHIFT, oh_first * g.sh - g.ph, n0 * g.C + c0, &bars[s]);
                if (two_imgs) tma_load_3d(st + p.xblock, &xmap, iw0 - SHIFT, -g.ph, (n0 + 1) * g.C + c0, &bars[s]);
                bulk_load(st + w_off, wt_k + (size_t)c0 * RS * TILE_K, p.w_stage * sizeof(float), &bars[s]);
                if (PAR) bulk_load(st + w2_off, wt2_k + (size_t)c0 * RS * TILE_K, p.w_stage * sizeof(float), &bars[s]);
                if (TWO) {
                    bulk_load(st + a_off, at_k + (size_t)c0 * TILE_K, p.ab_stage * sizeof(float), &bars[s]);
                    bulk_load(st + b_off, bt_k + (size_t)c0 * TILE_K, p.ab_stage * sizeof(float), &bars[s]);
                }
            }
        } else {
            // x halo tile: one warp per (channel, slot) row, lanes along the columns
            for (int cc = 0; cc < p.CC; ++cc) {
                const bool cok = (c0 + cc < g.C);
                const float* src_c = xg + (size_t)(cok ? c0 + cc : 0) * chw;
                float* dst_c = st + (size_t)cc * p.NSLOTS * p.XP;
                for (int sl = warp; sl < p.NSLOTS; sl += NWARPS) {
                    const int off = slot_off[sl];
                    const bool rok = cok && (off >= 0);
                    const float* src_row = src_c + (rok ? off : 0);
                    float* dst_row = dst_c + sl * p.XP;
                    for (int col = lane; col < p.XW; col += 32) {
                        const int iw = iw0 + col;
                        const bool ok = rok && iw >= 0 && iw < g.W;
                        if (!ok && g.neutral) dst_row[col] = pad_value(g, 0.0f);   // plain store, visible after the barrier
                        else cp_async4(dst_row + col, ok ? src_row + iw : xg, ok);
                    }
                }
            }
            // weights (and alpha, beta): contiguous blocks, 16 bytes per copy
            const float* wsrc = wt_k + (size_t)c0 * RS * TILE_K;
            for (int e = tid; e < p.w_stage / 4; e += NT) cp_async16(st + w_off + e * 4, wsrc + e * 4);
            if (PAR) {
                const float* wsrc2 = wt2_k + (size_t)c0 * RS * TILE_K;
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

    // accumulators
    float acc[TK][Q][4];   // Sum forms: running sum; Max/Min combine: running best
    int cbest[WIN && CHAN != CH_SUM ? TK : 1][Q][4];
#pragma unroll
    for (int k = 0; k < TK; ++k)
#pragma unroll
        for (int q = 0; q < Q; ++q)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[k][q][j] = (CHAN == CH_SUM) ? 0.0f : (CHAN == CH_MAX ? -INFINITY : INFINITY);
                if (WIN && CHAN != CH_SUM) cbest[k][q][j] = 0;
            }

    const size_t plane = (size_t)g.OH * g.OW;
    const size_t cplane = (size_t)g.OH * g.OWP;   // winner codes: rows padded to whole quads
    // Sum forms with winners: where this thread's codes of (its first output channel, input channel 0) go
    uint8_t* code_base[Q];
#pragma unroll
    for (int q = 0; q < Q; ++q) {
        code_base[q] = nullptr;
        if (WIN && CHAN == CH_SUM && out_row[q] >= 0) {
            const int n = out_row[q] / g.OH, oh = out_row[q] - n * g.OH;
            code_base[q] = reinterpret_cast<uint8_t*>(p.winners) +
                           (((size_t)n * g.K + (size_t)kt * TILE_K) * g.C * cplane + (size_t)oh * g.OWP + qcol[q]) *
                               (RS > 16 ? 2 : 1);
        }
    }
    const int row_step = g.dh * p.XP;
    const int chan_step = p.NSLOTS * p.XP;
    issue_chunk(0, 0);
    for (int ch = 0; ch < p.nchunks; ++ch) {
        const int s = ch & 1;
        float* st = stage0 + s * p.stage_floats;
        if (ch + 1 < p.nchunks) issue_chunk(ch + 1, s ^ 1);
        if constexpr (XTMA) {
            if (!mbar_wait(&bars[s], (ch >> 1) & 1)) {
                // the copy did not land in time: flag it, give the copies in flight one more
                // bounded chance to finish, and leave
                if (p.status) *p.status = 1;
                mbar_wait(&bars[s], (ch >> 1) & 1);
                if (ch + 1 < p.nchunks) mbar_wait(&bars[s ^ 1], ((ch + 1) >> 1) & 1);
                return;
            }
        } else {
            if (ch + 1 < p.nchunks) cp_async_wait<1>(); else cp_async_wait<0>();
            __syncthreads();
        }
        const float* ws = st + w_off + kg * TK;
        const float* ws2 = st + w2_off + kg * TK;
        const float* as = st + a_off + kg * TK;
        const float* bs = st + b_off + kg * TK;
        const int nc = min(p.CC, g.C - ch * p.CC);
        for (int cc = 0; cc < nc; ++cc) {
            // the R rows of input this thread's quads touch in channel cc
            float xr[Q][R][L];
#pragma unroll
            for (int q = 0; q < Q; ++q)
#pragma unroll
                for (int r = 0; r < R; ++r)
                    load_segment<SHIFT, L>(st + cc * chan_step + xoff[q] + r * row_step, xr[q][r]);
            const float* wc = ws + cc * (RS * TILE_K);
            const float* wc2 = ws2 + cc * (RS * TILE_K);

            if constexpr (WIN && CHAN == CH_SUM) {
                // Sum forms that emit winners.  Per pair of output channels and per pixel the RS tap
                // sums stay in registers, feed the extrema, and then give the winning taps on the
                // FMA pipe: with m the exact extremum, d = (t - m) * 2^32 is computed with one
                // rounding and is zero exactly for the taps that attain m;
                // key = |d| * (-2^125) + (2^23 + rank(tap)) equals 2^23 + rank for those taps and is
                // below 2^23 for every other tap, so the largest key belongs to the lowest winning
                // tap when rank decreases with the tap, and the low mantissa bits of that key are
                // rank itself: 15 - tap for the min branch (low nibble of the code), 16 * (15 - tap)
                // for the max branch (high nibble), both read back with one complement-and-mask.
                // (a non-zero |d| * 2^125 is at least 256 > 240, the largest rank; |x + w| < 2^95 is assumed.)
                // Windows above 16 taps use 16-bit codes: rank = 255 - tap (low byte) and
                // 256 * (255 - tap) (high byte); the scale grows to 2^41 so that a non-zero
                // |d| * 2^125 (at least 2^17) still exceeds every rank, |x + w| < 2^86 assumed.
                constexpr bool WIDE = RS > 16;
                constexpr int CW = WIDE ? 2 : 1;             // bytes per code
                constexpr int RTOP = WIDE ? 255 : 15, RMUL = WIDE ? 256 : 16;
                constexpr float kS = WIDE ? 2199023255552.0f : 4294967296.0f;   // 2^41 : 2^32
                constexpr float kH = 4.253529586511731e37f;  // 2^125
                constexpr float kB = 8388608.0f;             // 2^23
                constexpr bool DO_MIN = TWO || TAP_MIN, DO_MAX = TWO || !TAP_MIN;
                const int c = ch * p.CC + cc;
                float av[TK], bv[TK];
                if constexpr (TWO) {
                    loadn<TK>(as + cc * TILE_K, av);
                    loadn<TK>(bs + cc * TILE_K, bv);
                }
#pragma unroll
                for (int kp = 0; kp < TK / 2; ++kp) {
                    float wa[RS][2], wb[PAR ? RS : 1][2];
#pragma unroll
                    for (int tap = 0; tap < RS; ++tap) {
                        loadn<2>(wc + tap * TILE_K + 2 * kp, wa[tap]);
                        if constexpr (PAR) loadn<2>(wc2 + tap * TILE_K + 2 * kp, wb[tap]);
                    }
#pragma unroll
                    for (int q = 0; q < Q; ++q) {
                        unsigned packed[2] = {0u, 0u}, packed_hi[2] = {0u, 0u};   // 4 codes per channel (wide: two words)
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float ta[RS][2], tb[PAR ? RS : 1][2];
#pragma unroll
                            for (int tap = 0; tap < RS; ++tap) {
                                const float xv = xr[q][tap / S][j * SW + (tap % S) * DW];
                                add2(xv, wa[tap][0], wa[tap][1], ta[tap][0], ta[tap][1]);
                                if constexpr (PAR) add2(xv, wb[tap][0], wb[tap][1], tb[tap][0], tb[tap][1]);
                            }
                            const float (*tm)[2] = PAR ? tb : ta;   // sums of the max branch
                            unsigned bits_min[2] = {0u, 0u}, bits_max[2] = {0u, 0u};
                            float lo[2] = {0.0f, 0.0f}, hi[2] = {0.0f, 0.0f};
                            if constexpr (DO_MIN) {
                                lo[0] = fold_taps<RS>(ta, 0, true);
                                lo[1] = fold_taps<RS>(ta, 1, true);
                            }
                            if constexpr (DO_MAX) {
                                hi[0] = fold_taps<RS>(tm, 0, false);
                                hi[1] = fold_taps<RS>(tm, 1, false);
                            }
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                float& a = acc[2 * kp + h][q][j];
                                if constexpr (TWO) {
                                    a = __fmaf_rn(av[2 * kp + h], lo[h], a);
                                    a = __fmaf_rn(bv[2 * kp + h], hi[h], a);
                                } else {
                                    a = __fadd_rn(a, TAP_MIN ? lo[h] : hi[h]);
                                }
                            }
                            if constexpr (DO_MIN) {
                                const float e0 = -lo[0] * kS, e1 = -lo[1] * kS;
                                float key[RS][2];
#pragma unroll
                                for (int tap = 0; tap < RS; ++tap) {
                                    float d0 = e0, d1 = e1;
                                    fma2s(kS, ta[tap][0], ta[tap][1], d0, d1);             // >= 0
                                    key[tap][0] = key[tap][1] = kB + (float)(RTOP - tap);
                                    fma2s(-kH, d0, d1, key[tap][0], key[tap][1]);
                                }
                                bits_min[0] = __float_as_uint(fold_taps<RS>(key, 0, false));
                                bits_min[1] = __float_as_uint(fold_taps<RS>(key, 1, false));
                            }
                            if constexpr (DO_MAX) {
                                const float e0 = -hi[0] * kS, e1 = -hi[1] * kS;
                                float key[RS][2];
#pragma unroll
                                for (int tap = 0; tap < RS; ++tap) {
                                    float d0 = e0, d1 = e1;
                                    fma2s(kS, tm[tap][0], tm[tap][1], d0, d1);             // <= 0
                                    key[tap][0] = key[tap][1] = kB + (float)(RMUL * (RTOP - tap));
                                    fma2s(kH, d0, d1, key[tap][0], key[tap][1]);
                                }
                                bits_max[0] = __float_as_uint(fold_taps<RS>(key, 0, false));
                                bits_max[1] = __float_as_uint(fold_taps<RS>(key, 1, false));
                            }
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                unsigned code;
                                constexpr unsigned MLO = WIDE ? 0x00ffu : 0x0fu, MHI = WIDE ? 0xff00u : 0xf0u;
                                if constexpr (TWO) code = (~bits_min[h] & MLO) | (~bits_max[h] & MHI);
                                else code = TAP_MIN ? (~bits_min[h] & MLO) : (~bits_max[h] & MHI);
                                if constexpr (!WIDE) packed[h] |= code << (8 * j);
                                else if (j < 2) packed[h] |= code << (16 * j);
                                else packed_hi[h] |= code << (16 * (j - 2));
                            }
                        }
                        // one byte per (n, k, c, oh, ow): low nibble argmin tap, high nibble argmax tap
                        if (out_row[q] >= 0) {
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const int kl = kg * TK + 2 * kp + h;
                                if (kt * TILE_K + kl >= g.K) continue;
                                uint8_t* dst = code_base[q] + ((size_t)kl * g.C + c) * cplane * CW;
                                if (qcol[q] < g.OW) {   // the quad's 4 codes in one store (rows are padded)
                                    if constexpr (WIDE) *reinterpret_cast<uint2*>(dst) = make_uint2(packed[h], packed_hi[h]);
                                    else *reinterpret_cast<unsigned*>(dst) = packed[h];
                                }
                            }
                        }
                    }
                }
            } else {
            float mx[CARRIED ? 1 : TK][Q][4];           // per-channel extremum (max branch / single branch)
            float mn[TWO ? TK : 1][Q][4];               // per-channel minimum (two-branch modes)

            {
                // taps folded in groups: a fresh chain opens with 3 taps, later groups take 2
                constexpr int FIRST = CARRIED ? 2 : (RS >= 3 ? 3 : RS);
                constexpr int NG = 1 + (RS - FIRST + 1) / 2;
#pragma unroll
                for (int gi = 0; gi < NG; ++gi) {
                    const int t0 = (gi == 0) ? 0 : FIRST + 2 * (gi - 1);
                    const int nt = (gi == 0) ? (FIRST < RS ? FIRST : RS) : ((RS - t0) < 2 ? (RS - t0) : 2);
                    float wv[3][TK], wv2[PAR ? 3 : 1][TK];
#pragma unroll
                    for (int u = 0; u < 3; ++u)
                        if (u < nt) {
                            loadn<TK>(wc + (t0 + u) * TILE_K, wv[u]);
                            if constexpr (PAR) loadn<TK>(wc2 + (t0 + u) * TILE_K, wv2[u]);
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
                            for (int kp = 0; kp < TK / 2; ++kp) {
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
                float av[TK], bv[TK];
                if constexpr (TWO) {
                    loadn<TK>(as + cc * TILE_K, av);
                    loadn<TK>(bs + cc * TILE_K, bv);
                }
                const int c = ch * p.CC + cc;
#pragma unroll
                for (int k = 0; k < TK; ++k)
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
            }
            }
        }
        __syncthreads();  // every thread is done with this stage before it is refilled
    }

    // epilogue: bias, store, winner index of the Max / Min channel combines
    float* yg = reinterpret_cast<float*>(p.y);
    if constexpr (STATS) {
        // per-channel sums of the outputs and of their squares over this tile (the statistics a
        // following batch normalisation needs): per thread over its pixels, then a fixed shuffle
        // tree over the warp, which owns all pixels of the tile for its TK channels
        static_assert(PW == 1, "one warp per channel group owns the whole pixel tile");
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            const int kk = kt * TILE_K + kg * TK + k;
            const float bk = (p.bias && kk < g.K) ? p.bias[kk] : 0.0f;
            float s1 = 0.0f, s2 = 0.0f;
#pragma unroll
            for (int q = 0; q < Q; ++q)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float v = p.bias ? __fadd_rn(acc[k][q][j], bk) : acc[k][q][j];
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
        for (int k = 0; k < TK; ++k) {
            const int kk = kt * TILE_K + kg * TK + k;
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
                // extremum (same rounded adds as the main loop, so equality is exact)
                int32_t* idx = reinterpret_cast<int32_t*>(p.winners);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int ow = qcol[q] + j;
                    if (ow >= g.OW) continue;
                    const int c = cbest[k][q][j];
                    const float* xc = xg + ((size_t)n * g.C + c) * chw;
                    // the window's weights in their original layout: 9 adjacent values
                    const float* wk = reinterpret_cast<const float*>(p.w) + ((size_t)kk * g.C + c) * RS;
                    int tapw = 0;
#pragma unroll
                    for (int tap = RS - 1; tap >= 0; --tap) {
                        const int ih = oh * g.sh - g.ph + (tap / S) * g.dh;
                        const int iw = ow * SW - g.pw + (tap % S) * DW;
                        const float xv = (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) ? xc[(size_t)ih * g.W + iw] : pad_value(g, 0.0f);
                        if (__fadd_rn(xv, wk[tap]) == acc[k][q][j]) tapw = tap;
                    }
                    idx[o + j] = c * RS + tapw;
                }
            }
        }
    }
}

// ----------------------------------------------------------------------------------
// host side: tile selection and launch

// Failure-test switch (environment, read once): TCONV_DEBUG_DROP_COPY=1 makes the copy-engine
// kernels skip the copies of their first chunk, so that a test can watch a bounded wait run out with
// nothing in flight.  Unset / 0: off.
inline bool failure_test_switch() {
    static const bool v = [] {
        const char* e = getenv("TCONV_DEBUG_DROP_COPY");
        return e && e[0] == '1';
    }();
    return v;
}

struct TiledPlan {
    TiledParams p;
    dim3 grid;
    int threads;
    size_t smem;
    int tile_k;
    bool xtma;
    size_t ws_w, ws_ab;  // workspace split (bytes): each weight array, each of alpha / beta
};

inline size_t tiled_ws_bytes(const Geo& g) {
    // upper bound over every tile choice: K padded to 64, C padded to the chunk size (8, 6 or 4)
    const size_t Kp = ((size_t)g.K + 63) / 64 * 64, Cp = (size_t)g.C + 7;
    const size_t w = Kp * Cp * g.RS * sizeof(float);
    const size_t ab = Kp * Cp * sizeof(float);
    return 2 * w + 2 * ab + 1024;
}

inline int round_up(int v, int a) { return (v + a - 1) / a * a; }

// One candidate plan: ragged tiles allowed or not, cc input channels per staged chunk.
template <int R, int S, int SW, int DW, int Q, int KG, int PW, int TK = 8>
inline bool plan_tiles_opt(const Geo& g, bool par, bool two, int esize, bool allow_ragged, int cc, TiledPlan* pl) {
    TiledParams& p = pl->p;
    constexpr int TILE_K = KG * TK;
    constexpr int NQ = Q * 32 * PW;
    const int qpr_full = (g.OW + 3) / 4;
    // column tiles: at most NQ/4 quads wide (a tile keeps >= 4 rows unless the row is short), split evenly
    const int max_qpr = NQ >= 32 ? NQ / 4 : NQ;
    const int ncol = (qpr_full + max_qpr - 1) / max_qpr;
    p.QPR = (qpr_full + ncol - 1) / ncol;
    // every column tile must start on a 16-byte boundary of the input row (TMA): with 2-byte
    // elements that needs an even number of 8-byte quads per tile
    if (esize == 2 && ncol > 1 && ((p.QPR * SW) & 1)) p.QPR += 1;
    p.TW = p.QPR * 4;
    p.n_col_tiles = (g.OW + p.TW - 1) / p.TW;
    p.TH = NQ / p.QPR;
    if (p.TH < 1) return false;
    p.total_rows = g.N * g.OH;
    p.total_quads = p.total_rows * p.QPR;
    p.xblock = 0;
    // rows whose quads do not divide the lanes: tiles of NQ consecutive quads of the flattened
    // (n, oh, quad) space instead of whole rows, so that every lane owns a quad
    p.ragged = (allow_ragged && ncol == 1 && NQ % p.QPR != 0 && p.total_quads > NQ) ? 1 : 0;
    const int rows_max = p.ragged ? (p.QPR - 1 + NQ - 1) / p.QPR + 1 : p.TH;   // rows one tile can touch
    // TMA path: rows of x are 16-byte multiples, "same" padding along w (fixes the column shift),
    // and tiles that stay inside one image without idling more than a quarter of the lanes
    // (ragged tiles: inside two images, each staged by its own copy)
    const int unit = 16 / esize;                                     // elements per 16 bytes
    const int shift = esize == 4 ? TmaShift<S, DW, 4>::value : TmaShift<S, DW, 2>::value;
    const int th_img = p.TH < g.OH ? p.TH : g.OH;
    const int tiles_img = (g.OH + th_img - 1) / th_img;
    const bool rows_fit = p.ragged ? (g.OH * p.QPR >= NQ)
                                   : ((double)g.OH / (tiles_img * th_img) >= 0.75 && th_img * p.QPR * 4 >= NQ * 3);
    // (a bf16 layer fed with float x converts while staging element by element: no tensor copy)
    pl->xtma = !g.xf32 && ((g.W * esize) % 16 == 0) && (g.pw == (S - 1) * DW / 2) && rows_fit;
    p.XW = (p.TW - 1) * SW + (S - 1) * DW + 1;   // == (QPR-1)*4*SW + L
    if (pl->xtma && p.ragged) {
        p.TH = rows_max;
        p.tiles_per_img = 0;
        p.n_row_tiles = (p.total_quads + NQ - 1) / NQ;
        p.GAP = 0;
        p.NSLOTS = (rows_max - 1) * g.sh + (R - 1) * g.dh + 1;
        p.XP = round_up(p.XW + shift, unit);
        if (p.XP > 256 || p.NSLOTS > 256) return false;
    } else if (pl->xtma) {
        p.TH = th_img;
        p.tiles_per_img = tiles_img;
        p.n_row_tiles = g.N * tiles_img;
        p.GAP = 0;
        p.NSLOTS = (p.TH - 1) * g.sh + (R - 1) * g.dh + 1;
        p.XP = round_up(p.XW + shift, unit);
        if (p.XP > 256 || p.NSLOTS > 256) return false;
    } else {
        if (p.ragged) p.TH = rows_max;
        if (p.TH > p.total_rows) p.TH = p.total_rows;
        p.tiles_per_img = 0;
        p.n_row_tiles = p.ragged ? (p.total_quads + NQ - 1) / NQ : (p.total_rows + p.TH - 1) / p.TH;
        p.GAP = (R - 1) * g.dh - g.sh + 1;
        if (p.GAP < 0) p.GAP = 0;
        const int max_imgs = (p.TH - 1) / g.OH + 2;
        p.NSLOTS = (p.TH - 1) * g.sh + (R - 1) * g.dh + 1 + (max_imgs - 1) * p.GAP;
        p.XP = round_up(p.XW, unit);
    }
    p.CC = cc;
    p.Cpad = round_up(g.C, p.CC);
    p.nchunks = p.Cpad / p.CC;
    // one stage: x tile | weights | (weights 2) | alpha | beta, each block 128-byte aligned;
    // sizes in 4-byte words (XP counts elements of esize bytes)
    p.xbox = p.CC * p.NSLOTS * p.XP;
    p.xblock = round_up(p.xbox, 128 / esize);
    p.x_stage = round_up(((pl->xtma && p.ragged) ? p.xblock + p.xbox : p.xbox) * esize / 4, 32);
    p.w_stage = p.CC * g.RS * TILE_K;            // multiple of 32 floats
    p.ab_stage = two ? p.CC * TILE_K : 0;
    p.stage_floats = p.x_stage + p.w_stage * (par ? 2 : 1) + 2 * p.ab_stage;
    pl->smem = 2 * (size_t)p.stage_floats * sizeof(float) + 16 + (size_t)p.NSLOTS * sizeof(int) + 16;
    // 2-byte elements without TMA: a table of source offsets for one channel plane of the tile
    if (!pl->xtma && esize == 2) pl->smem += ((size_t)p.NSLOTS * p.XP + 4) * sizeof(int);
    if (pl->smem > 200 * 1024) return false;
    const int nkt = (g.K + TILE_K - 1) / TILE_K;
    pl->grid = dim3((unsigned)(p.n_col_tiles * p.n_row_tiles), (unsigned)nkt, 1);
    pl->threads = KG * PW * 32;
    pl->tile_k = TILE_K;
    pl->ws_w = (size_t)nkt * p.Cpad * g.RS * TILE_K * sizeof(float);
    pl->ws_ab = (size_t)nkt * p.Cpad * TILE_K * sizeof(float);
    return true;
}

// Picks the plan: ragged tiles keep every lane busy but stage taller (and, with TMA, two) input
// blocks; the first candidate whose two stages leave room for four resident CTAs per SM wins, in
// the order ragged / whole rows, 8 / 4 channels per chunk; else whole rows with 8 channels.
template <int R, int S, int SW, int DW, int Q, int KG, int PW, int TK = 8>
inline bool plan_tiles(const Geo& g, bool par, bool two, int esize, TiledPlan* pl) {
    // 8 channels per chunk when four CTAs stay resident, else 4 channels when three do (measured
    // on the stride-2 56 -> 28 layer: 8.06 against 7.86 Ttap/s for whole-row tiles at four CTAs)
    // (two-branch kernels with 8 channels per thread hold two CTAs per SM by their registers: their
    // stages may use half of the shared memory)
    const bool two_resident = two && TK == 8;
    for (int cc = 8; cc >= 4; cc -= 2) {
        const size_t budget = (two_resident ? 112 : (cc == 4 ? 74 : 56)) * 1024;
        TiledPlan cand = *pl;
        if (plan_tiles_opt<R, S, SW, DW, Q, KG, PW, TK>(g, par, two, esize, true, cc, &cand) && cand.p.ragged &&
            cand.smem <= budget) {
            *pl = cand;
            return true;
        }
    }
    return plan_tiles_opt<R, S, SW, DW, Q, KG, PW, TK>(g, par, two, esize, false, 8, pl);
}

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);

inline encode_tiled_fn get_encode_tiled() {
    static encode_tiled_fn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            f = nullptr;
        return (encode_tiled_fn)f;
    }();
    return fn;
}

// x viewed as [N*C][H][W]; box = [CC][NSLOTS][XP]; out-of-range elements read as the padding value.
// The encoded map is a pure function of the arguments below, so the last few are kept per host
// thread (a training loop calls each layer with the same buffers step after step).
struct XMapKey {
    const void* x;
    long long nc;
    int W, H, esize, XP, NSLOTS, CC, neutral;
};
constexpr int kXMapCache = 16;

inline bool encode_x_map(const Geo& g, const void* x, int esize, const TiledParams& p, CUtensorMap* map);

inline bool make_x_map(const Geo& g, const void* x, int esize, const TiledParams& p, CUtensorMap* map) {
    static thread_local XMapKey keys[kXMapCache];
    static thread_local CUtensorMap maps[kXMapCache];
    static thread_local int used = 0, next = 0;
    XMapKey k;
    memset(&k, 0, sizeof(k));
    k.x = x; k.nc = (long long)g.N * g.C; k.W = g.W; k.H = g.H; k.esize = esize;
    k.XP = p.XP; k.NSLOTS = p.NSLOTS; k.CC = p.CC; k.neutral = g.neutral;
    for (int i = 0; i < used; ++i)
        if (memcmp(&keys[i], &k, sizeof(k)) == 0) {
            *map = maps[i];
            return true;
        }
    if (!encode_x_map(g, x, esize, p, map)) return false;
    keys[next] = k;
    maps[next] = *map;
    next = (next + 1) % kXMapCache;
    if (used < kXMapCache) ++used;
    return true;
}

inline bool encode_x_map(const Geo& g, const void* x, int esize, const TiledParams& p, CUtensorMap* map) {
    encode_tiled_fn enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.N * g.C};
    const cuuint64_t strides[2] = {(cuuint64_t)g.W * esize, (cuuint64_t)g.H * g.W * esize};
    const cuuint32_t box[3] = {(cuuint32_t)p.XP, (cuuint32_t)p.NSLOTS, (cuuint32_t)p.CC};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUtensorMapDataType dt = esize == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    // out-of-range elements: zeros (zero padding) or NaN (neutral padding: min / max skip a NaN)
    return enc(map, dt, 3, const_cast<void*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               g.neutral ? CU_TENSOR_MAP_FLOAT_OOB_FILL_NAN_REQUEST_ZERO_FMA : CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Arguments of one forward launch (host side).
struct FwdArgs {
    Geo g;
    int dtype;
    float* stats;      // NULL, or where the tiled kernel leaves its per-tile channel statistics
    size_t stats_bytes;
    int stats_tiles;   // out: tiles the kernel wrote (0: the kernel that ran wrote none)
    int stats_k;       // out: channel pitch of the partials
    const void *x, *w, *w2;
    const float *alpha, *beta, *bias;
    void* y;
    void* winners;
    void* ws;
    size_t ws_bytes;
    int* status;
    cudaStream_t st;
    const char* name;  // out: kernel variant
};

template <typename T, int MODE, int CHAN, bool WIN, int R, int S, int SW, int DW, int Q, int KG, int PW, int TK>
int launch_tiled_variant(FwdArgs& a) {
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    constexpr bool PAR = (MODE == TCONV_PARALLEL);
    const Geo& g = a.g;
    TiledPlan pl;
    pl.p.g = g;
    if (!plan_tiles<R, S, SW, DW, Q, KG, PW, TK>(g, PAR, TWO, (int)sizeof(T), &pl)) return TCONV_ERR_UNSUPPORTED;
    const size_t need = pl.ws_w * (PAR ? 2 : 1) + (TWO ? 2 * pl.ws_ab : 0);
    if (!a.ws || a.ws_bytes < need) return TCONV_ERR_WORKSPACE_TOO_SMALL;
    float* wt = reinterpret_cast<float*>(a.ws);
    float* wt2 = PAR ? wt + pl.ws_w / sizeof(float) : nullptr;
    float* at = TWO ? wt + (pl.ws_w * (PAR ? 2 : 1)) / sizeof(float) : nullptr;
    float* bt = TWO ? at + pl.ws_ab / sizeof(float) : nullptr;
    CUtensorMap xmap;
    memset(&xmap, 0, sizeof(xmap));
    if (pl.xtma && !make_x_map(g, a.x, (int)sizeof(T), pl.p, &xmap)) return TCONV_ERR_CUDA;
    const int nkt = pl.grid.y;
    const size_t nrep = (size_t)nkt * pl.p.Cpad * g.RS * pl.tile_k;
    repack_weights_kernel<T><<<(unsigned)((nrep + 255) / 256), 256, 0, a.st>>>(
        g.K, g.C, g.RS, pl.tile_k, pl.p.Cpad, nkt, (const T*)a.w, (const T*)a.w2, a.alpha, a.beta, wt, wt2, at, bt);
    pl.p.x = a.x; pl.p.w = a.w; pl.p.wt = wt; pl.p.wt2 = wt2; pl.p.at = at; pl.p.bt = bt;
    pl.p.bias = a.bias; pl.p.y = a.y; pl.p.winners = a.winners; pl.p.status = a.status;
    // channel statistics in the epilogue: winner-emitting kernels (the training forward); a call
    // without winners takes them from the stored output afterwards (stats_tiles stays 0)
    pl.p.stats = nullptr; pl.p.stats_k = nkt * pl.tile_k;
    if (a.stats && WIN) {
        if ((size_t)pl.grid.x * pl.p.stats_k * 2 * sizeof(float) > a.stats_bytes) return TCONV_ERR_WORKSPACE_TOO_SMALL;
        pl.p.stats = a.stats; a.stats_tiles = (int)pl.grid.x; a.stats_k = pl.p.stats_k;
    }
    pl.p.debug_drop = failure_test_switch();
#define TCONV_LAUNCH_F32_S(XTMAV, RAGV, STATSV)                                                       \
    {                                                                                                \
        auto kern = fwd_tiled_f32_kernel<MODE, CHAN, WIN, XTMAV, RAGV, R, S, SW, DW, Q, KG, PW, TK, STATSV>; \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) \
            return TCONV_ERR_CUDA;                                                                   \
        kern<<<pl.grid, pl.threads, pl.smem, a.st>>>(xmap, pl.p);                                    \
    }
#define TCONV_LAUNCH_F32(XTMAV, RAGV)                                                                 \
    {                                                                                                \
        if constexpr (WIN) { if (pl.p.stats) TCONV_LAUNCH_F32_S(XTMAV, RAGV, true) else TCONV_LAUNCH_F32_S(XTMAV, RAGV, false) } \
        else TCONV_LAUNCH_F32_S(XTMAV, RAGV, false)                                                  \
    }
    if (pl.xtma) {
        if (pl.p.ragged) TCONV_LAUNCH_F32(true, true) else TCONV_LAUNCH_F32(true, false)
        a.name = WIN ? "fwd_tiled_f32_tma_win" : "fwd_tiled_f32_tma";
    } else {
        if (pl.p.ragged) TCONV_LAUNCH_F32(false, true) else TCONV_LAUNCH_F32(false, false)
        a.name = WIN ? "fwd_tiled_f32_win" : "fwd_tiled_f32";
    }
#undef TCONV_LAUNCH_F32
#undef TCONV_LAUNCH_F32_S
    return TCONV_OK;
}

// Geometry families with a tiled kernel: 3x3 windows with (stride_w, dil_w) in
// {(1,1), (2,1), (1,2), (1,4)}, and the 1 x 3 and 5 x 5 windows at stride 1, dilation 1.
template <typename T, int MODE, int CHAN, bool WIN>
int launch_tiled_geom(FwdArgs& a) {
    constexpr bool TWO = (MODE == TCONV_COMPOUND || MODE == TCONV_PARALLEL);
    // two quads per thread where one running value per output suffices (the carried
    // extremum of layers (iv), (v) without winners), else one
    constexpr bool CARRIED = !TWO && !WIN && ((MODE == TCONV_MAX_PLUS && CHAN == CH_MAX) ||
                                              (MODE == TCONV_MIN_PLUS && CHAN == CH_MIN));
    constexpr int Q = CARRIED ? kQuadsCarried : 1;
    // Sum forms that emit winners work on one pair of output channels at a time: 4 channels per
    // thread (2 or 8 measured no faster); two-branch kernels keep three values per output: 4 channels per thread leave room for
    // four resident CTAs per SM (measured 3-6 % faster than 8 channels per thread)
    constexpr int TK = (WIN && CHAN == CH_SUM) ? 4 : (TWO ? 4 : 8);
    const Geo& g = a.g;
    if (g.R == 3 && g.S == 3) {
        if (g.sw == 1 && g.dw == 1) return launch_tiled_variant<T, MODE, CHAN, WIN, 3, 3, 1, 1, Q, 4, 1, TK>(a);
        // stride 2: the longer input segments of a quad are amortised over 8 channels per thread
        // in the winner-free two-branch kernels (measured +3 % on the 56 -> 28 layer)
        constexpr int TK2 = (TWO && !WIN) ? 8 : TK;
        if (g.sw == 2 && g.dw == 1) return launch_tiled_variant<T, MODE, CHAN, WIN, 3, 3, 2, 1, Q, 4, 1, TK2>(a);
        if (g.sw == 1 && g.dw == 2) return launch_tiled_variant<T, MODE, CHAN, WIN, 3, 3, 1, 2, Q, 4, 1, TK>(a);
        if (g.sw == 1 && g.dw == 4) return launch_tiled_variant<T, MODE, CHAN, WIN, 3, 3, 1, 4, Q, 4, 1, TK>(a);
    }
    // the other windows of the paper's networks: 1 x 3 (1-D layers as signals of unit height) and 5 x 5
    if (g.R == 1 && g.S == 3 && g.sw == 1 && g.dw == 1)
        return launch_tiled_variant<T, MODE, CHAN, WIN, 1, 3, 1, 1, Q, 4, 1, TK>(a);
    if (g.R == 5 && g.S == 5 && g.sw == 1 && g.dw == 1)
        return launch_tiled_variant<T, MODE, CHAN, WIN, 5, 5, 1, 1, Q, 4, 1, TK>(a);
    return TCONV_ERR_UNSUPPORTED;
}

// One instance per (mode, channel combine): compiled in its own translation unit.
template <int MODE, int CHAN>
int launch_fwd_tiled_inst(FwdArgs& a) {
    if (a.dtype != TCONV_F32) return TCONV_ERR_UNSUPPORTED;  // bf16: separate kernel
    // (windows above 16 taps: the Sum forms emit 16-bit codes)
    if ((double)a.g.N * a.g.C * a.g.H * a.g.W >= 2.0e9) return TCONV_ERR_UNSUPPORTED;  // 32-bit offsets
    if (a.winners) return launch_tiled_geom<float, MODE, CHAN, true>(a);
    return launch_tiled_geom<float, MODE, CHAN, false>(a);
}

}  // namespace tconv

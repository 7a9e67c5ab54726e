// Shared device/host definitions of the tropical-convolution kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tconv.h"

namespace tconv {

// Channel combine after TCONV_CHAN_DEFAULT has been resolved.
enum { CH_SUM = 1, CH_MAX = 2, CH_MIN = 3 };

// Layer geometry as the kernels see it (plain ints, passed by value).
struct Geo {
    int N, C, H, W, K, R, S;
    int sh, sw, ph, pw, dh, dw;
    int OH, OW, RS;
    int OWP;         // OW rounded up to a multiple of 4: row pitch of the Sum-form winner codes
    int mode, chan;  // tconv_mode_t, resolved channel combine
    int wide;        // Sum-form winner codes are uint16 (R*S > 16) instead of uint8
    int neutral;     // padded taps hold NaN, which min / max skip (neutral padding), instead of zero
    int xf32;        // bf16 layer whose x is float: rounded to bf16 while it is staged
};

// Value a padded tap reads: zero, or a quiet NaN under neutral padding (min.f32 / max.f32 and their
// bf16x2 forms return the other operand when one is NaN, so the tap never takes part).
__device__ __forceinline__ float pad_value(const Geo& g, float) { return g.neutral ? __int_as_float(0x7fc00000) : 0.0f; }
__device__ __forceinline__ __nv_bfloat16 pad_value(const Geo& g, __nv_bfloat16) {
    return __ushort_as_bfloat16((unsigned short)(g.neutral ? 0x7fc0 : 0));
}

__host__ __device__ inline bool two_branch(int mode) {
    return mode == TCONV_COMPOUND || mode == TCONV_PARALLEL;
}

// One tap sum in the layer's arithmetic type, returned as float (a bf16 value
// converts exactly).  fp32: one rounded add.  bf16: one rounded bf16 add.
__device__ __forceinline__ float tap_add(float x, float w) { return __fadd_rn(x, w); }
__device__ __forceinline__ float tap_add(__nv_bfloat16 x, __nv_bfloat16 w) {
    return __bfloat162float(__hadd(x, w));
}

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
    return __float2bfloat16_rn(v);
}

template <typename T> __device__ __forceinline__ T zero_of();
template <> __device__ __forceinline__ float zero_of<float>() { return 0.0f; }
template <> __device__ __forceinline__ __nv_bfloat16 zero_of<__nv_bfloat16>() {
    return __float2bfloat16_rn(0.0f);
}

// Deterministic block-wide sum (fixed tree): every thread passes its partial,
// thread 0 receives the total.  `red` holds blockDim.x floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
    const int tid = threadIdx.x;
    red[tid] = v;
    __syncthreads();
    for (int step = blockDim.x >> 1; step > 0; step >>= 1) {
        if (tid < step) red[tid] += red[tid + step];
        __syncthreads();
    }
    float total = red[0];
    __syncthreads();
    return total;
}

}  // namespace tconv

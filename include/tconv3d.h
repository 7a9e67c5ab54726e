/*
 * tconv3d.h - C ABI of the three-dimensional tropical convolution layers (sm_100a).
 *
 * The operations are the three-dimensional extension of the paper's Section 3.2 (base operators
 * MinPlus3d / MaxPlus3d: min / max over the T x R x S window of x + w, and the six Conv3d
 * layers (i)-(vi) that take Sum, Max or Min of a base operator over the input channels) and the
 * Conv3d forms of the compound layer (section "Compound tropical convolution layers": sum over c of alpha * MinPlus3d + beta *
 * MaxPlus3d of one weight, the two branches sharing each addition) and of the parallel layer
 * (section "Parallel tropical convolution layers": weight w in the min branch, w2 in the max branch).
 *
 * Conventions (the same as tconv.h, which provides the enums and status codes used here):
 *   - every pointer is a DEVICE pointer unless stated; descriptors and sizes live on the host;
 *   - dense tensors, PyTorch Conv3d layout: x[N][C][D][H][W], w / w2 [K][C][T][R][S],
 *     y / grad_y [N][K][OD][OH][OW], alpha / beta fp32 [K][C], bias fp32 [K]; the paper's
 *     definition is symmetric in the three spatial axes, "depth" names the slowest one;
 *   - zero padding takes part in min / max as x = 0; output extents follow PyTorch;
 *   - ties go to the lowest flattened (c, t, r, s); the two-branch combine is
 *     fmaf(alpha, min, acc) then fmaf(beta, max, acc) in fp32, channels ascending; bias last;
 *   - bf16 layers: every tap sum is one rounded bf16 add, the channel combine is fp32, y is
 *     rounded once;
 *   - calls enqueue work on `stream` (a cudaStream_t passed as void*) and return without
 *     synchronising; the caller owns every buffer and keeps it alive until the stream has run;
 *   - results are deterministic: no atomics, fixed summation order for a given build;
 *   - return value: TCONV_OK or a negative tconv_status_t; nothing is launched on an error
 *     found by the host-side checks.  T*R*S must not exceed 256, and every tensor must have
 *     fewer than 2^31 elements.
 */
#ifndef TCONV3D_H
#define TCONV3D_H

#include "tconv.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tconv3d_desc_t {
    int32_t N, C, D, H, W; /* input  [N][C][D][H][W]                   */
    int32_t K, T, R, S;    /* weight [K][C][T][R][S]                   */
    int32_t stride_d, stride_h, stride_w;
    int32_t pad_d, pad_h, pad_w;
    int32_t dil_d, dil_h, dil_w;
    int32_t mode;          /* tconv_mode_t                              */
    int32_t chan;          /* tconv_chan_t; compound / parallel: sum    */
    int32_t dtype;         /* tconv_dtype_t of x, w, w2, y, grad_y, grad_x */
} tconv3d_desc_t;

/* Output extents.  Host call. */
int tconv3d_output_shape(const tconv3d_desc_t *desc, int32_t *OD, int32_t *OH, int32_t *OW);

/*
 * Bytes of the winner buffer, 0 for an invalid descriptor.  Layout:
 *   Max / Min channel combine: int32 [N][K][OD][OH][OW], value c*T*R*S + (t*R + r)*S + s;
 *   Sum channel combine (incl. compound, parallel): uint16 [N][K][C][OD][OH][OW], argmin tap in
 *     the low byte, argmax tap in the high byte; a single-branch layer fills only its own byte.
 */
size_t tconv3d_winner_bytes(const tconv3d_desc_t *desc);

/* Scratch bytes tconv3d_backward needs (backward = 1; covers winners == NULL); the forward
 * pass (backward = 0) needs none.  Host call. */
size_t tconv3d_workspace_bytes(const tconv3d_desc_t *desc, int backward);

/*
 * Forward pass of one layer.  w2: max-branch weights (parallel mode), else NULL.  alpha, beta:
 * compound / parallel only, NULL means all ones.  bias may be NULL.  winners: NULL, or a buffer of
 * tconv3d_winner_bytes() that receives the winning taps for tconv3d_backward.
 */
int tconv3d_forward(const tconv3d_desc_t *desc, const void *x, const void *w, const void *w2,
                    const float *alpha, const float *beta, const float *bias, void *y,
                    void *winners, void *stream);

/*
 * Backward pass: grad_y goes wholly to the winner(s) of every output.  winners: the buffer the
 * forward pass filled for the same inputs, or NULL to have it recomputed into the workspace.
 * grad_x [N][C][D][H][W] in the descriptor's dtype (fp32 accumulation; winners inside the padding
 * contribute nothing); grad_w, grad_w2 fp32 [K][C][T][R][S] (grad_w2: max branch of parallel
 * mode); grad_alpha, grad_beta fp32 [K][C] (sum of grad_y * MinPlus3d resp. MaxPlus3d);
 * grad_bias fp32 [K].  Any gradient pointer may be NULL.  workspace: at least
 * tconv3d_workspace_bytes(desc, 1) bytes, 256-byte aligned.
 */
int tconv3d_backward(const tconv3d_desc_t *desc, const void *x, const void *w, const void *w2,
                     const float *alpha, const float *beta, const void *grad_y, const void *winners,
                     void *grad_x, float *grad_w, float *grad_w2, float *grad_alpha, float *grad_beta,
                     float *grad_bias, void *workspace, size_t workspace_bytes, void *stream);

/* Kernels launched so far by this thread's tconv3d_* calls (for launch accounting). */
long long tconv3d_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TCONV3D_H */

/*
 * tconv.h - C ABI of the B200 tropical-convolution library (libtconv.so).
 *
 * Operators (paper: "Compound and Parallel Modes of Tropical Convolutional
 * Neural Networks"):
 *   - base operators MinPlus2d / MaxPlus2d, Section 3.1: min / max over the
 *     R x S window of x[n, c, ih, iw] + w[k, c, r, s];
 *   - the six TCNN layers (i)-(vi), Section 3.1: Sum, Max or Min of the base
 *     operator over the input channels c;
 *   - the compound layer, section "Compound tropical convolution layers":
 *       y = sum_c ( alpha[k,c] * MinPlus2d(x, w) + beta[k,c] * MaxPlus2d(x, w) ),
 *     both branches sharing one addition per tap;
 *   - the parallel layer, section "Parallel tropical convolution layers": the same with w in the min branch and
 *     w2 in the max branch;
 *   - backward: the upstream gradient is routed wholly to the winning tap(s).
 *
 * Conventions the paper leaves open and this library fixes:
 *   - geometry follows the PyTorch convolution convention (cross-correlation,
 *     OH = floor((H + 2*pad_h - dil_h*(R-1) - 1) / stride_h) + 1, input row
 *     ih = oh*stride_h - pad_h + r*dil_h);
 *   - padding is zero padding by default: a padded tap takes part in min / max as x = 0;
 *     with pad_mode = TCONV_PAD_NEUTRAL a padded tap holds the identity of its branch's
 *     semiring (+inf under min, -inf under max: section "Tropical algebra and tropical
 *     convolution"), i.e. it never wins;
 *   - ties go to the lowest flattened (c, r, s); channels are combined in
 *     ascending order, in fp32, compound/parallel as
 *       acc = fmaf(alpha, min_c, acc); acc = fmaf(beta, max_c, acc);
 *   - one bias[k], added last.
 *
 * Every pointer is a DEVICE pointer unless stated otherwise, dense, row-major,
 * 16-byte aligned, owned by the caller.  The library never allocates or frees
 * device memory; scratch space comes from the caller's workspace.  Calls are
 * asynchronous on the given stream (a cudaStream_t passed as void*, NULL = the
 * default stream).  Outputs are overwritten, never accumulated into.
 *
 * Every function that returns int returns TCONV_OK (0) or a negative
 * tconv_status_t; nothing throws, aborts or prints.  Non-finite inputs are
 * outside the contract.  Winner codes of the fp32 Sum forms (incl. compound and
 * parallel) are recovered from scaled differences of tap sums: they are exact for
 * |x + w| < 2^95 (windows of up to 16 taps) and |x + w| < 2^86 (larger windows);
 * beyond that the outputs y are still exact but winners may be wrong.  There is no
 * CPU implementation behind this interface.
 */
#ifndef TCONV_H
#define TCONV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TCONV_MAX_PLUS = 0, /* MaxPlus2d base operator (Section 3.1)            */
    TCONV_MIN_PLUS = 1, /* MinPlus2d base operator (Section 3.1)            */
    TCONV_COMPOUND = 2, /* compound layer (CompoundMinMaxPlusSumConv2d2p), Sum over channels */
    TCONV_PARALLEL = 3  /* parallel layer (ParallelMinMaxPlusSumConv2d2p), Sum over channels */
} tconv_mode_t;

typedef enum {
    TCONV_CHAN_DEFAULT = 0, /* MAX for max_plus, MIN for min_plus, SUM otherwise */
    TCONV_CHAN_SUM = 1,     /* layers (i), (ii); the only choice for compound / parallel */
    TCONV_CHAN_MAX = 2,     /* layers (iii), (v) */
    TCONV_CHAN_MIN = 3      /* layers (iv), (vi) */
} tconv_chan_t;

typedef enum {
    TCONV_F32 = 0, /* x, w, w2, y, grad_y, grad_x are float                          */
    TCONV_BF16 = 1 /* they are bf16; each tap sum is one bf16 add; the channel
                      combine, alpha, beta, bias and parameter gradients stay fp32 */
} tconv_dtype_t;

typedef enum {
    TCONV_PAD_ZERO = 0,   /* padded taps take part in min / max as x = 0 */
    TCONV_PAD_NEUTRAL = 1 /* padded taps are skipped (semiring identity); every window must keep at
                             least one tap inside the image, else TCONV_ERR_UNSUPPORTED; dense 2-D
                             entry points only */
} tconv_pad_mode_t;

typedef enum {
    TCONV_X_SAME = 0, /* x has the descriptor's dtype */
    TCONV_X_F32 = 1   /* dtype = TCONV_BF16 only: x is float and is rounded to bf16 (nearest even)
                         while it is staged, bit-identical to converting x first; grad_x stays bf16 */
} tconv_x_dtype_t;

typedef enum {
    TCONV_OK = 0,
    TCONV_ERR_INVALID_ARG = -1,         /* NULL descriptor / required pointer, non-positive size    */
    TCONV_ERR_UNSUPPORTED = -2,         /* e.g. compound with a Max/Min channel combine, R*S > 256 */
    TCONV_ERR_MISALIGNED = -3,          /* a tensor pointer is not 16-byte aligned                  */
    TCONV_ERR_WORKSPACE_TOO_SMALL = -4, /* workspace_bytes below tconv_workspace_bytes()            */
    TCONV_ERR_CUDA = -5,                /* launch failed; text in tconv_last_error()                */
    TCONV_ERR_DEVICE_TIMEOUT = -6,      /* a bounded device-side wait gave up (tconv_device_status) */
    TCONV_ERR_TOO_LARGE = -7            /* a size exceeds what the entry point supports             */
} tconv_status_t;

/* Layer geometry.  x is [N][C][H][W], w and w2 are [K][C][R][S], y and grad_y
 * are [N][K][OH][OW], alpha and beta are [K][C], bias is [K]. */
typedef struct {
    int32_t N, C, H, W; /* input batch, channels, height, width */
    int32_t K, R, S;    /* output channels, window height, window width */
    int32_t stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
    int32_t mode;  /* tconv_mode_t  */
    int32_t chan;  /* tconv_chan_t  */
    int32_t dtype; /* tconv_dtype_t */
    int32_t pad_mode; /* tconv_pad_mode_t */
    int32_t x_dtype;  /* tconv_x_dtype_t  */
} tconv_desc_t;

/* Output extent of the layer (PyTorch convention, Section 5).  Host call. */
int tconv_output_shape(const tconv_desc_t *desc, int32_t *OH, int32_t *OW);

/*
 * Size in bytes of the winner buffer of a layer, 0 if the descriptor is
 * invalid.  Layout:
 *   Max / Min channel combine: int32 [N][K][OH][OW], value c*R*S + r*S + s;
 *   Sum channel combine (incl. compound, parallel): one code per
 *     (n, k, c, oh, ow), laid out [N][K][C][OH][OWP] with the row pitch
 *     OWP = OW rounded up to a multiple of 4 (the codes of a row's columns
 *     OW..OWP-1 are padding: tconv_forward fills them with valid taps and
 *     tconv_backward relies on that); uint8 with the argmin
 *     tap r*S+s in the low nibble and the argmax tap in the high nibble when
 *     R*S <= 16, else uint16 with the argmin tap in the low byte and the argmax
 *     tap in the high byte (R*S <= 256).  A single-branch Sum layer fills only
 *     its own half; the other half is 0.
 */
size_t tconv_winner_bytes(const tconv_desc_t *desc);

/*
 * Scratch bytes tconv_forward (backward = 0) or tconv_backward (backward = 1)
 * needs.  For the backward pass the figure covers the case winners == NULL
 * (winners recomputed into the workspace).  Host call.
 */
size_t tconv_workspace_bytes(const tconv_desc_t *desc, int backward);

/*
 * Forward pass of one layer (sections "Tropical algebra and tropical convolution", "Compound tropical convolution layers",
 * "Parallel tropical convolution layers").
 *   x, w        inputs and weights (dtype of the descriptor).
 *   w2          max-branch weights, parallel mode only; NULL otherwise.
 *   alpha, beta fp32 [K][C], compound / parallel only; NULL means all ones
 *               (the parameter-free variant); ignored by max_plus / min_plus.
 *   bias        fp32 [K] or NULL.
 *   y           output (dtype of the descriptor); bf16 outputs are rounded to
 *               nearest even from the fp32 result.
 *   winners     NULL, or a buffer of tconv_winner_bytes() that receives the
 *               winning taps (layout above) for a later tconv_backward.
 *   workspace   scratch of at least tconv_workspace_bytes(desc, 0) bytes; may
 *               be NULL when that is 0.
 */
int tconv_forward(const tconv_desc_t *desc, const void *x, const void *w, const void *w2,
                  const float *alpha, const float *beta, const float *bias, void *y,
                  void *winners, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Forward pass that also returns the per-channel statistics of its output,
 *   sum_y[k]  = sum over (n, oh, ow) of y[n][k][oh][ow],
 *   sum_y2[k] = sum over (n, oh, ow) of y[n][k][oh][ow]^2      (fp32 [K] each),
 * i.e. what the batch normalisation that follows every tropical layer in the paper's
 * residual blocks (section "ResNet Models": Conv-BN-Tropical-BN and Tropical-BN-Tropical-BN)
 * needs for its mean and variance, without reading y again.  The sums are taken over the
 * stored values (bf16 layers: after rounding) in the kernel's epilogue: per pixel tile with a
 * fixed shuffle tree, then over the tiles in a fixed order (deterministic, no atomics).  Other
 * arguments and results as tconv_forward; workspace_bytes must be at least
 * tconv_stats_workspace_bytes(desc).
 */
size_t tconv_stats_workspace_bytes(const tconv_desc_t *desc);
int tconv_forward_stats(const tconv_desc_t *desc, const void *x, const void *w, const void *w2,
                        const float *alpha, const float *beta, const float *bias, void *y,
                        void *winners, float *sum_y, float *sum_y2, void *workspace,
                        size_t workspace_bytes, void *stream);

/*
 * Backward pass: routes grad_y to the winner(s) of every output.
 *   winners     the buffer tconv_forward filled for the same inputs, or NULL to
 *               have the winners recomputed (into the workspace).
 *   grad_x      [N][C][H][W] in the descriptor's dtype (fp32 accumulation);
 *               taps that won inside the padding contribute nothing here.
 *   grad_w      fp32 [K][C][R][S]; in parallel mode the min branch only.
 *   grad_w2     fp32 [K][C][R][S], parallel mode (max branch); NULL otherwise.
 *   grad_alpha, grad_beta  fp32 [K][C], compound / parallel:
 *               sum over (n, oh, ow) of grad_y * MinPlus2d resp. * MaxPlus2d.
 *   grad_bias   fp32 [K].
 * Any gradient pointer may be NULL: that gradient is skipped.  Gradients are
 * deterministic: no atomics, fixed summation order for a given build.
 */
int tconv_backward(const tconv_desc_t *desc, const void *x, const void *w, const void *w2,
                   const float *alpha, const float *beta, const void *grad_y,
                   const void *winners, void *grad_x, float *grad_w, float *grad_w2,
                   float *grad_alpha, float *grad_beta, float *grad_bias, void *workspace,
                   size_t workspace_bytes, void *stream);

/*
 * Forward pass for callers that cannot allocate device memory.  (The paper has no
 * counterpart of this entry point; it exists for the library's users.)
 *
 * Some callers have no way to hand over a workspace: code that runs where the CUDA
 * allocator must not be touched (a real-time loop that was given a fixed memory budget
 * at start-up), plug-ins whose host application owns all device memory, and small C
 * programs that link this library without a tensor framework.  For them this variant of tconv_forward takes
 * its scratch (the repacked weights, alpha and beta of the tiled kernels) from a fixed
 * array inside the library image instead of a caller workspace.  It calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *
 *   - Arguments are those of tconv_forward without workspace / workspace_bytes; the
 *     caller still owns and passes every input and output.
 *   - The built-in scratch holds tconv_forward_noalloc_max_scratch() bytes (8 MiB; every
 *     GPU that loads the library holds that much until the process exits).  A layer with
 *     tconv_workspace_bytes(desc, 0) above that is rejected with TCONV_ERR_TOO_LARGE and
 *     a message in tconv_last_error(); nothing is launched.
 *   - The first call on each device looks up the device address of the scratch (with
 *     that device current).  Make that first call before starting any stream capture.
 *   - All calls share the one array.  Each call rewrites every byte of it that it later
 *     reads, so nothing depends on earlier contents; but two calls whose kernels overlap
 *     on the GPU (different streams, or different host threads) race on it.  Serialise
 *     them on one stream or with events.
 * Results are identical to tconv_forward's.
 */
int tconv_forward_noalloc(const tconv_desc_t *desc, const void *x, const void *w, const void *w2,
                          const float *alpha, const float *beta, const float *bias, void *y,
                          void *winners, void *stream);

/* Capacity in bytes of the scratch tconv_forward_noalloc uses.  Host call. */
size_t tconv_forward_noalloc_max_scratch(void);

/*
 * Depthwise form (groups = C): every channel is its own group, the arrangement the paper's
 * MobileNetV2 variants use when they replace the depthwise convolutions (Section 6, "MobileNetV2
 * Models"):
 *   y[n][c] = alpha[c] * min_tap(x[n][c] + w[c]) + beta[c] * max_tap(x[n][c] + w2[c]) + bias[c]
 * (compound: w2 = w; max_plus / min_plus: the one extremum, no alpha / beta).  The descriptor is the
 * dense one with K == C (else TCONV_ERR_INVALID_ARG) and R * S <= 16 (else TCONV_ERR_UNSUPPORTED);
 * chan is ignored (a group has one channel).  Shapes: x, grad_x [N][C][H][W]; y, grad_y
 * [N][C][OH][OW]; w, w2, grad_w, grad_w2 [C][R][S]; alpha, beta, bias and their gradients [C].
 * winners: uint8 [N][C][OH][OW], argmin tap r*S+s in the low nibble, argmax tap in the high nibble
 * (tconv_dw_winner_bytes() bytes).  Tie rule, padding, evaluation order, bf16 semantics, NULL alpha /
 * beta / bias and error behaviour are those of tconv_forward / tconv_backward; every result equals
 * the dense layer with one input and one output channel applied channel by channel.
 * tconv_dw_forward needs no workspace; y may be NULL when only the winners are wanted.
 * tconv_dw_backward needs tconv_dw_workspace_bytes(desc, 1) bytes (recomputed winners when
 * winners == NULL, and the per-chunk partial sums of the parameter gradients); any gradient pointer
 * may be NULL; gradients are deterministic (gather form for grad_x, fixed-order reductions).
 * Layers whose element counts exceed 2^31 - 1 are rejected with TCONV_ERR_TOO_LARGE.
 */
size_t tconv_dw_winner_bytes(const tconv_desc_t *desc);
size_t tconv_dw_workspace_bytes(const tconv_desc_t *desc, int backward);
int tconv_dw_forward(const tconv_desc_t *desc, const void *x, const void *w, const void *w2,
                     const float *alpha, const float *beta, const float *bias, void *y,
                     void *winners, void *stream);
int tconv_dw_backward(const tconv_desc_t *desc, const void *x, const void *w, const void *w2,
                      const float *alpha, const float *beta, const void *grad_y,
                      const void *winners, void *grad_x, float *grad_w, float *grad_w2,
                      float *grad_alpha, float *grad_beta, float *grad_bias, void *workspace,
                      size_t workspace_bytes, void *stream);

/*
 * Number of operations the paper's complexity analysis (Section 4.1) assigns to
 * one forward pass of the layer: additions + comparisons + multiplications
 * (theta = 1).  Host call; 0 for an invalid descriptor.
 */
double tconv_paper_ops(const tconv_desc_t *desc);

/*
 * Register-only throughput probe of the plain ALUs: every thread of a full-GPU
 * grid runs `iters` rounds of independent add + max/min chains in the
 * instruction mix `variant` (see tconv_alu_probe_name), with no memory traffic,
 * and one result is written to `sink` (device, >= 4 bytes) so the work cannot be
 * elided.  *taps_per_launch (host) receives the number of tropical taps
 * (one x + w term folded into its running min and/or max) one launch performs.
 * Used to measure the add+max/min roofline the kernels are compared against.
 */
int tconv_alu_probe(int variant, int iters, void *sink, double *taps_per_launch, void *stream);

/* Name of probe variant i, NULL past the last one.  Host call. */
const char *tconv_alu_probe_name(int variant);

/*
 * Device-side health check.  The kernels wait for their asynchronous copies with a
 * bounded number of polls; a wait that gives up sets a status word on the device and
 * the kernel returns early (its outputs are then undefined).  This call synchronises
 * `stream`, reads the word, clears it, and returns TCONV_OK or
 * TCONV_ERR_DEVICE_TIMEOUT.
 */
int tconv_device_status(void *stream);

/* Text for a status code.  Host call. */
const char *tconv_status_string(int status);

/* Text of the last CUDA error this thread's calls met ("" if none).  Host call. */
const char *tconv_last_error(void);

/* Name of the kernel variant the last tconv_forward / tconv_backward of this
 * thread launched (for benchmark records).  Host call. */
const char *tconv_last_kernel(void);

/* Number of GPU kernels the calling thread's calls into this library have launched so
 * far (cumulative).  Host call. */
long long tconv_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TCONV_H */

/*
 * hq.h -- C ABI of the B200 (sm_100a) Hadamard-quantized layer forward.
 *
 * The operations are the ones HQ-DM states for a quantized linear / convolution layer:
 *   online Hadamard transform of the activations (Eq. 10, with H_k of Eq. 5-7)
 *   -> symmetric quantization to N-bit integer codes with a floating-point scale (Eq. 3)
 *   -> integer matrix product / convolution with offline-prepared integer weights (Eq. 12, Eq. 14)
 *   -> rescale by S_XH * S_W in front of the integer product (Eq. 12, Eq. 14), plus bias.
 *
 * Conventions (all entry points):
 *   - Return value is an hq_status; nothing throws, prints or allocates device memory.
 *   - "device" pointers are CUDA device addresses owned by the caller for the duration of
 *     the asynchronous work; "host" pointers are ordinary process memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Work is enqueued
 *     asynchronously on it; a non-OK status means nothing was launched.
 *   - Activations are row-major [rows][cols] with the channel (reduction) axis contiguous;
 *     convolution activations are NHWC.  Weights are [N][RS][C] (output channel, filter tap,
 *     input channel), i.e. the transpose of the paper's W in R^{Ci x Co}.
 *   - Row pitches ("ld*") are in ELEMENTS for floating-point tensors and in BYTES for code
 *     tensors.  Base pointers and pitches of code / output tensors must be 16-byte aligned.
 *   - dev_status (optional, may be NULL) is a device int32 the kernels set to a non-zero
 *     word if a bounded on-chip wait expired; copy it to the host and pass it to
 *     hq_check_status.  It is never cleared by the library.
 */
#ifndef HQ_H_
#define HQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif
/* The library is built with hidden visibility (two builds loaded into one process must not bind to one another's
 * internals); the entry points declared here are its only exported symbols. */
#if defined(__GNUC__)
#pragma GCC visibility push(default)
#endif

typedef enum {
    HQ_OK = 0,
    HQ_ERR_INVALID_ARG = 1,   /* NULL where a pointer is required, unknown enum value */
    HQ_ERR_SHAPE = 2,         /* sizes that contradict each other (cols % had_block, K mismatch ...) */
    HQ_ERR_UNSUPPORTED = 3,   /* legal request the library has no kernel for */
    HQ_ERR_ALIGNMENT = 4,     /* pointer or pitch not aligned as stated above */
    HQ_ERR_WORKSPACE = 5,     /* workspace too small (ask hq_workspace_size) */
    HQ_ERR_OVERFLOW_RISK = 6, /* int32 accumulators could overflow for these bit-widths and K */
    HQ_ERR_CUDA = 7,          /* a CUDA runtime / driver call failed (launch, tensor-map encode) */
    HQ_ERR_TIMEOUT = 8,       /* a bounded device-side wait expired (reported via dev_status) */
    HQ_ERR_SCRATCH_LIMIT = 9  /* hq_qlinear_noalloc: the layer needs more than the library's built-in scratch */
} hq_status;

typedef enum { HQ_F32 = 0, HQ_BF16 = 1 } hq_dtype;

/* Storage of activation codes.  NIBBLE: two codes per byte, element 2j in the low nibble, 2j+1 in
 * the high nibble, two's complement (3-bit codes are sign-extended to a nibble).  INT8: one code per byte. */
typedef enum { HQ_CODES_NIBBLE = 0, HQ_CODES_INT8 = 1 } hq_container;

/* PER_ROW: one dynamic scale per row (token / pixel), S = max|xH| / qmax.  STATIC: one scalar for
 * the whole tensor, read from device memory (the learned per-timestep scale of the paper). */
typedef enum { HQ_SCALE_PER_ROW = 0, HQ_SCALE_STATIC = 1 } hq_scale_mode;

/* How the offline weight integers are formed.
 *  PLAIN : B = Q(W)                       (Eq. 3 per output channel)
 *  FOLDED: B = H_raw * Q(W)               (the inner product of Eq. 12 / Eq. 14, exact integers; the
 *                                          paper's Single-Hadamard semantics; needs w_bits + log2(had_block) bits)
 *  DOUBLE: B = Q(H^T W), H orthonormal    (the Double-Hadamard scheme the paper compares against)
 *  PLAIN_A2: B = Q(W) laid out for activations that arrive as TWO int8 limbs per channel, [hi(C) | lo(C)] per pixel
 *            (the width-axis convolution with blocks wider than 16 positions, whose integer activations q * H_raw need
 *            more than 8 bits): the blob describes 2C input channels per tap and two weight limbs, "hi" rows
 *            [Q(W) | 0] and "lo" rows [0 | Q(W)], so that the two-limb product 256 * acc_hi + acc_lo of the kernel is
 *            sum (256 * a_hi + a_lo) * Q(W). */
typedef enum { HQ_W_PLAIN = 0, HQ_W_FOLDED = 1, HQ_W_DOUBLE = 2, HQ_W_PLAIN_A2 = 3 } hq_weight_mode;

/* Host-side description of a prepared weight blob (filled by hq_weight_prepare). */
typedef struct {
    int64_t N;          /* output channels */
    int64_t C;          /* input channels per tap */
    int32_t RS;         /* filter taps (1 for a linear layer, 9 for 3x3) */
    int32_t w_bits;     /* 4 or 8 */
    int32_t had_block;  /* 2^k, or <= 1 for no transform */
    int32_t mode;       /* hq_weight_mode */
    int32_t limbs;      /* 1: B fits a signed byte; 2: B = 256*hi + lo, lo in [-128,127] */
    int32_t container;  /* hq_container of the activation codes this blob pairs with (fixes the byte order along K) */
    int64_t C_pad;      /* C rounded up to the kernel's K tile (128); padding is zero */
    int64_t N_pad;      /* N rounded up to 128; padding rows are zero */
    int64_t bytes;      /* size of the blob */
    int32_t max_abs_b;  /* largest |B| entry, for the accumulator-range check */
    int32_t reserved;
} hq_weight_desc;

int hq_version(void);
const char* hq_status_string(hq_status s);

/* Decode a dev_status word the caller copied back to the host: HQ_OK if zero, else HQ_ERR_TIMEOUT. */
hq_status hq_check_status(const int32_t* dev_status_host_copy);

/* ---- Eq. 10 + Eq. 3: codes = Q(x * BlockDiag(H_k)) ------------------------------------------------
 * x          device, [rows][cols] of xdt, pitch ldx elements (16-byte aligned rows).
 * had_block  2^k dividing cols (Eq. 10: cols = m * 2^k), or 0/1 for H = I (the bypass after Eq. 10).
 * bits       3, 4 or 8.  NIBBLE container needs bits <= 4 and cols even.
 * mode       PER_ROW: scales[rows] is written, S = max_j |(xH)_j| / qmax(bits), H orthonormal (the
 *            2^(-k/2) of Eq. 7 is inside S); an all-zero row gets S = 1.
 *            STATIC : static_scale (device, 1 float) is read; scales[0] (if scales != NULL) receives a copy.
 * codes      device, [rows] x ld_codes bytes; code = clamp(rint(xH / S), -2^(bits-1), 2^(bits-1)-1), ties to even.
 * Errors: NULL pointers, cols % had_block, had_block not a power of two -> no launch. */
hq_status hq_hadamard_quant(const void* x, hq_dtype xdt, int64_t rows, int64_t cols, int64_t ldx,
                            int had_block, int bits, hq_scale_mode mode, const float* static_scale,
                            void* codes, hq_container cont, int64_t ld_codes, float* scales, void* stream);

/* ---- Offline weight side (host code, not timed): Eq. 3 per output channel, then the chosen mode. ----
 * w          host fp32 [N][RS][C].
 * container  the activation container the blob will be multiplied with.
 * blob       host buffer of hq_weight_blob_bytes(...) bytes; copy it to the device as is.
 * s_w        host [N] per-output-channel scales (for DOUBLE: scales of H^T W).
 * desc       filled on success.
 * Errors: FOLDED/DOUBLE with C % had_block != 0; FOLDED whose integers need more than 2 limbs -> HQ_ERR_OVERFLOW_RISK. */
int64_t hq_weight_blob_bytes(int64_t N, int32_t RS, int64_t C, int32_t w_bits, int32_t had_block,
                             hq_weight_mode mode);
hq_status hq_weight_prepare(const float* w, int64_t N, int32_t RS, int64_t C, int32_t w_bits, int32_t had_block,
                            hq_weight_mode mode, hq_container container, void* blob, int64_t blob_bytes,
                            float* s_w, hq_weight_desc* desc);

/* ---- Eq. 12: integer product + rescale ------------------------------------------------------------
 * acc[m][o] = sum_k a[m][k] * B[o][k]  (int32, exact);  y = alpha * S_a[m] * S_w[o] * acc + bias[o].
 * a_codes    device, [M] x lda bytes, container and a_bits as produced by hq_hadamard_quant.
 * desc/w_dev host descriptor and device copy of the blob; desc->RS must be 1 and desc->C == K.
 * scale_a    device [M], or [1] if scale_a_is_scalar.  scale_w device [N].  bias device [N] or NULL.
 * alpha      2^(-k/2) for FOLDED weights with had_block = 2^k, else 1 (hq_alpha_for computes it).
 * acc_out    device int32 [M][N] (pitch N) or NULL.   y: device [M] x ldy elements of ydt, or NULL.
 * Errors: K mismatch, container mismatch with the blob, accumulator bound K * qmax_a * max|B| >= 2^31
 * -> HQ_ERR_OVERFLOW_RISK. */
hq_status hq_qgemm(const void* a_codes, hq_container cont, int a_bits, int64_t M, int64_t K, int64_t lda,
                   const hq_weight_desc* desc, const void* w_dev, const float* scale_a, int scale_a_is_scalar,
                   const float* scale_w, const float* bias, float alpha, int32_t* acc_out, void* y,
                   hq_dtype ydt, int64_t ldy, int32_t* dev_status, void* stream);

/* ---- Eq. 14 (transform on the channel axis): integer convolution + rescale --------------------------
 * a_codes NHWC [Nb][H][W] x (C codes, densely packed); weights [Cout][R][S][C] inside the blob; R = S in {1,3},
 * stride in {1,2}, pad in {0,1}; zero padding.  Output NHWC [Nb][Ho][Wo][Cout], Ho = (H + 2 pad - R)/stride + 1.
 * scale_a_is_scalar != 0: y = alpha * S_a * S_w[o] * acc + bias[o].
 * scale_a_is_scalar == 0: scale_a is [Nb*H*W], one per INPUT pixel, and each tap is rescaled by the scale of
 *   the pixel it read: y = alpha * S_w[o] * sum_taps S_a[pix(tap)] * acc_tap + bias[o]. */
hq_status hq_qconv2d(const void* a_codes, hq_container cont, int a_bits, int64_t Nb, int64_t H, int64_t W,
                     int64_t C, const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                     const float* scale_a, int scale_a_is_scalar, const float* scale_w, const float* bias,
                     float alpha, int32_t* acc_out, void* y, hq_dtype ydt, int32_t* dev_status, void* stream);

/* ---- Fused layer: transform -> quantize -> integer product -> rescale in one call (Eq. 12 / Eq. 14). ----
 * Codes and scales live in `workspace` (device, hq_workspace_size bytes); the code container is desc->container.
 * alpha is derived from the descriptor.  y pitch ldy elements.
 * The product kernel is launched so that it may begin (set-up, first weight tile) while the transform kernel is still
 * running; it waits for the transform before it touches codes or activation scales.  Work enqueued on the stream before
 * the call has completed before either kernel starts, as usual. */
hq_status hq_workspace_size(int64_t rows, int64_t cols, hq_container cont, size_t* bytes);
hq_status hq_qlinear(const void* x, hq_dtype xdt, int64_t M, int64_t K, int64_t ldx, const hq_weight_desc* desc,
                     const void* w_dev, const float* scale_w, const float* bias, int a_bits, hq_scale_mode mode,
                     const float* static_scale, void* y, hq_dtype ydt, int64_t ldy, void* workspace,
                     size_t ws_bytes, int32_t* dev_status, void* stream);
hq_status hq_qconv(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                   const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                   const float* scale_w, const float* bias, int a_bits, hq_scale_mode mode,
                   const float* static_scale, void* y, hq_dtype ydt, void* workspace, size_t ws_bytes,
                   int32_t* dev_status, void* stream);

/* ---- The fused linear layer as ONE kernel: the transform and the quantization run inside the product kernel and write
 * their codes straight into the shared-memory operand tile the tensor core reads (the "online" transform of the
 * Single-Hadamard schematic, Eq. 10 -> Eq. 3 -> Eq. 12, without a trip of the codes through memory).  No workspace.
 * Same arithmetic and results as hq_qlinear.  Covers K in {128, 256, 512} (the whole reduction in one operand tile),
 * had_block in 32 .. K, weights prepared for the INT8 container, bf16 output with a 16-byte aligned pitch; anything else
 * returns HQ_ERR_UNSUPPORTED (use hq_qlinear). */
hq_status hq_qlinear_fused(const void* x, hq_dtype xdt, int64_t M, int64_t K, int64_t ldx, const hq_weight_desc* desc,
                           const void* w_dev, const float* scale_w, const float* bias, int a_bits, hq_scale_mode mode,
                           const float* static_scale, void* y, int64_t ldy, int32_t* dev_status, void* stream);

/* ---- Eq. 13 + Eq. 14 with the transform on the WIDTH axis, as the paper states the convolution ---------------------
 * The paper reshapes X_c [B][Cin][h][w] to (B*Cin*h) x w and multiplies by the block-diagonal H_c (w x w): every
 * image row of every channel is transformed along w.  The weights are quantized untransformed and the integer core
 * is Conv((X~ H_c)_int * H_c, W_int) with ONE activation scale in front (a per-row scale would not factor out of the
 * sum over channels and taps).
 *
 * hq_hadamard_quant_width: x device NHWC [Nb][H][W][C] (densely packed, C % 4 == 0) ->
 *   z = clamp(rint(x H_c / S)) * H_raw   as int8 NHWC (device), the integer activations of the convolution, and
 *   scale_out[0] = S * 2^(-k/2) (device, may be NULL), the scale that goes in front of it.
 *   had_block_w = 2^k divides W (0/1: no transform); static_scale = S (device, 1 float); bits in {3,4,8}.
 *   The integer factor must fit a signed byte: had_block_w * 2^(bits-1) <= 128 (16 positions at 4 bits, 32 at 3 bits),
 *   otherwise HQ_ERR_OVERFLOW_RISK.
 * hq_hadamard_quant_width2: the same for wider blocks (up to 64 positions, so the full width of a 32- or 64-wide feature
 *   map is one block as in Eq. 13): z is written as two int8 limbs per channel, z = 256 * hi + lo with lo in [-128, 127],
 *   z_limbs device NHWC [Nb][H][W][2C] = [hi(C) | lo(C)] per pixel.  C % 2 == 0.
 * hq_qconv_width: the whole layer.  desc / w_dev: PLAIN one-limb weights prepared for the INT8 container
 *   (had_block of the descriptor is ignored); workspace as for hq_qconv with the INT8 container;
 *   y = 2^(-k/2) * S * S_w[o] * Conv(z, W_int) + bias[o].  With a PLAIN_A2 descriptor (desc->C == 2 C) the layer runs
 *   through hq_hadamard_quant_width2 and the two-limb product; workspace hq_workspace_size(Nb*H*W, 2C, INT8). */
hq_status hq_hadamard_quant_width(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                  int had_block_w, int bits, const float* static_scale, void* z_codes,
                                  float* scale_out, void* stream);
hq_status hq_hadamard_quant_width2(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                                   int had_block_w, int bits, const float* static_scale, void* z_limbs,
                                   float* scale_out, void* stream);
hq_status hq_qconv_width(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                         const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                         const float* scale_w, const float* bias, int a_bits, int had_block_w,
                         const float* static_scale, void* y, hq_dtype ydt, void* workspace, size_t ws_bytes,
                         int32_t* dev_status, void* stream);

/* ---- LayerNorm with a per-sample affine fused in front of the transform + quantization (no counterpart in the paper's
 * equations: the "modulate(norm(x), shift, scale)" that precedes the quantized linears of a diffusion-transformer block;
 * the row statistics are taken from the registers that hold the row for the transform, so the activations make one trip
 * through memory). --------------------------------------------------------------------------------------------------
 * x        device [rows][ldx] fp32/bf16.   Per row: mean and biased variance over the cols values,
 *          y = (x - mean) / sqrt(var + eps) * weight[g][c] + bias[g][c],   g = row / rows_per_group
 *          (rows_per_group = 0: one vector pair for all rows).  For adaLN pass weight = 1 + scale, bias = shift.
 * weight, bias   device [groups][cols] fp32, 16-byte aligned, or NULL (1 and 0).   The rest as hq_hadamard_quant.
 * Restrictions: the row shapes of the fast kernel only (had_block in 32..4096, cols / 32 (64 above 512-wide blocks)
 * <= 256 threads per row and a CTA of at most 320 threads; 16-byte aligned codes and pitches), else HQ_ERR_UNSUPPORTED;
 * rows_per_group must be a multiple of the rows one CTA takes (any multiple of 32 is). */
hq_status hq_ln_quant(const void* x, hq_dtype xdt, int64_t rows, int64_t cols, int64_t ldx, const float* weight,
                      const float* bias, int64_t rows_per_group, float eps, int had_block, int bits,
                      hq_scale_mode mode, const float* static_scale, void* codes, hq_container cont,
                      int64_t ld_codes, float* scales, void* stream);

/* The fused layer with that prologue: LayerNorm + affine -> transform -> quantize (one activation scale per row) ->
 * integer product -> rescale.  Arguments as hq_ln_quant and hq_qlinear. */
hq_status hq_ln_qlinear(const void* x, hq_dtype xdt, int64_t M, int64_t K, int64_t ldx, const float* ln_weight,
                        const float* ln_bias, int64_t rows_per_group, float eps, const hq_weight_desc* desc,
                        const void* w_dev, const float* scale_w, const float* bias, int a_bits, void* y, hq_dtype ydt,
                        int64_t ldy, void* workspace, size_t ws_bytes, int32_t* dev_status, void* stream);

/* ---- GroupNorm + SiLU fused in front of the transform + quantization (no counterpart in the paper's equations:
 * the normalisation and activation that precede the quantized 3x3 convolutions of a UNet ResBlock, applied while the
 * activations are read, so that they make one trip through memory instead of three). ---------------------------------
 * x        device NHWC [Nb][H][W][C] fp32/bf16, densely packed.
 * groups   groups of C/groups consecutive channels (a multiple of 4 each); statistics per (sample, group) over
 *          H*W*(C/groups) values: y = (x - mean) / sqrt(var + eps) * gamma[c] + beta[c]; then y * sigmoid(y).
 * gamma, beta  device [C].   The rest as hq_hadamard_quant with rows = Nb*H*W, cols = C (transform over channels).
 * pre_bias device bf16 [Nb][C], 8-byte aligned, or NULL: a per-sample, per-channel addend (the projected step
 *          embedding of a residual block) that is added to x BEFORE the normalisation -- the statistics are those of
 *          x + pre_bias -- without the sum ever being written: the statistics pass adds it as it reads, and the
 *          quantize pass folds it into its per-channel offset.  Read only.
 * scratch  device, 16-byte aligned, Nb * groups * 24 bytes: fp64 sums (cleared by the call) and the statistics.
 * Restrictions: had_block in 32..4096 with at most 320 threads per CTA shape (else HQ_ERR_UNSUPPORTED), and the
 * rows of a sample must be a multiple of the rows one CTA takes (any H*W that is a multiple of 32 is). */
hq_status hq_gn_silu_quant(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C, int groups,
                           const float* gamma, const float* beta, const void* pre_bias, float eps, int had_block, int bits,
                           hq_scale_mode mode, const float* static_scale, void* codes, hq_container cont,
                           int64_t ld_codes, float* scales, void* scratch, size_t scratch_bytes, void* stream);

/* The fused convolution layer with that prologue: GroupNorm + SiLU -> transform -> quantize -> integer convolution ->
 * rescale.  Arguments as hq_gn_silu_quant and hq_qconv. */
hq_status hq_gn_silu_qconv(const void* x, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C, int groups,
                           const float* gamma, const float* beta, const void* pre_bias, float eps, const hq_weight_desc* desc,
                           const void* w_dev, int R, int S, int stride, int pad, const float* scale_w,
                           const float* bias, int a_bits, hq_scale_mode mode, const float* static_scale, void* y,
                           hq_dtype ydt, void* workspace, size_t ws_bytes, void* scratch, size_t scratch_bytes,
                           int32_t* dev_status, void* stream);


/* ---- The same calls on the channel concatenation of two tensors, read in place (no counterpart in the paper's
 * equations: the skip connections of the UNet join the up-sampling path by concatenation, and the concatenated tensor is
 * consumed only by quantized layers, so it need never be written).  x holds channels / columns [0, C1) (pitch C1, for
 * hq_hadamard_quant_cat ldx), x2 the channels [C1, C) (pitch C - C1, resp. ldx2); C1 must be a multiple of the Hadamard
 * block (a block never straddles the two tensors) and of 8, both tensors 16-byte aligned.  Everything else as the call
 * without `_cat`; the results are bit-identical to it applied to the written-out concatenation. */
hq_status hq_hadamard_quant_cat(const void* x, int64_t ldx, const void* x2, int64_t ldx2, int64_t cols1, hq_dtype xdt,
                                int64_t rows, int64_t cols, int had_block, int bits, hq_scale_mode mode,
                                const float* static_scale, void* codes, hq_container cont, int64_t ld_codes, float* scales,
                                void* stream);
hq_status hq_gn_silu_quant_cat(const void* x, const void* x2, int64_t C1, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W,
                               int64_t C, int groups, const float* gamma, const float* beta, const void* pre_bias,
                               float eps, int had_block, int bits, hq_scale_mode mode, const float* static_scale,
                               void* codes, hq_container cont, int64_t ld_codes, float* scales, void* scratch,
                               size_t scratch_bytes, void* stream);
hq_status hq_gn_silu_qconv_cat(const void* x, const void* x2, int64_t C1, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W,
                               int64_t C, int groups, const float* gamma, const float* beta, const void* pre_bias,
                               float eps, const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                               const float* scale_w, const float* bias, int a_bits, hq_scale_mode mode,
                               const float* static_scale, void* y, hq_dtype ydt, void* workspace, size_t ws_bytes,
                               void* scratch, size_t scratch_bytes, int32_t* dev_status, void* stream);
hq_status hq_qconv_cat(const void* x, const void* x2, int64_t C1, hq_dtype xdt, int64_t Nb, int64_t H, int64_t W, int64_t C,
                       const hq_weight_desc* desc, const void* w_dev, int R, int S, int stride, int pad,
                       const float* scale_w, const float* bias, int a_bits, hq_scale_mode mode, const float* static_scale,
                       void* y, hq_dtype ydt, void* workspace, size_t ws_bytes, int32_t* dev_status, void* stream);

/* ---- Fused linear layer with GroupNorm (optionally + SiLU) in front, on the pixels of an NHWC tensor: the QKV
 * projection of an attention block (no counterpart in the paper's equations; the paper quantizes the projection, the
 * normalisation in front of it is the network's own).  Rows = Nb * rows_per_sample; statistics per (sample, group) over
 * rows_per_sample * (C / groups) values; one activation scale per row.  Other arguments as hq_gn_silu_qconv / hq_qlinear. */
hq_status hq_gn_qlinear(const void* x, hq_dtype xdt, int64_t Nb, int64_t rows_per_sample, int64_t C, int groups,
                        const float* gamma, const float* beta, float eps, int silu, const hq_weight_desc* desc,
                        const void* w_dev, const float* scale_w, const float* bias, int a_bits, void* y, hq_dtype ydt,
                        int64_t ldy, void* workspace, size_t ws_bytes, void* scratch, size_t scratch_bytes,
                        int32_t* dev_status, void* stream);

/* ==== The unquantized operations between the quantized layers of the noise-prediction network ======================
 * The method replaces every linear and convolution of the network (overview figure of the framework; Experiments: the
 * first and last convolution stay in floating point); what follows is the arithmetic left between them.  None of it is
 * one of the paper's equations.  All tensors are device bf16 unless stated, channel axis contiguous, 16-byte aligned,
 * channel counts multiples of 8; every call is asynchronous on `stream` and returns an hq_status as above. */

/* out[i] = x[i] * sigmoid(x[i]); count elements (multiple of 8).  out may alias x. */
hq_status hq_silu(const void* x, int64_t count, void* out, void* stream);
/* out[i] = a[i] + b[i] (residual connections); out may alias a or b. */
hq_status hq_add(const void* a, const void* b, int64_t count, void* out, void* stream);
/* h[n][r][c] += e[n][c] in place: h [Nb][rows_per_sample][C], e [Nb][C] (the step/class embedding added to every pixel
 * of a sample inside a residual block). */
hq_status hq_add_rows_bcast(void* h, const void* e, int64_t Nb, int64_t rows_per_sample, int64_t C, void* stream);
/* emb[n][:] += table[labels[n]][:]: emb [Nb][dim], table [classes][dim], labels device int32 [Nb] (clamped to the table). */
hq_status hq_class_embed_add(void* emb, const void* table, const int32_t* labels, int64_t Nb, int64_t dim,
                             int64_t classes, void* stream);
/* Sinusoidal embedding of the denoising step: t device fp32 [Nb]; out [Nb][dim], dim even;
 * out[n][i] = cos(t[n] f_i), out[n][dim/2 + i] = sin(t[n] f_i), f_i = max_period^(-i / (dim/2)). */
hq_status hq_timestep_embedding(const float* t, int64_t Nb, int64_t dim, float max_period, void* out, void* stream);
/* Nearest-neighbour up-sampling by two: x NHWC [Nb][H][W][C] -> out [Nb][2H][2W][C]. */
hq_status hq_upsample_nearest2x(const void* x, int64_t Nb, int64_t H, int64_t W, int64_t C, void* out, void* stream);
/* Channel concatenation (skip connections): out[r] = a[r] | b[r], a [rows][Ca], b [rows][Cb], out [rows][Ca + Cb]. */
hq_status hq_concat_channels(const void* a, int64_t Ca, const void* b, int64_t Cb, int64_t rows, void* out,
                             void* stream);
/* GroupNorm as a pass of its own, with SiLU when silu != 0 (the normalisation in front of the unquantized last
 * convolution): x, out NHWC; gamma, beta device fp32 [C]; scratch as for hq_gn_silu_quant (Nb * groups * 24 bytes). */
hq_status hq_groupnorm_act(const void* x, int64_t Nb, int64_t H, int64_t W, int64_t C, int groups, const float* gamma,
                           const float* beta, float eps, int silu, void* out, void* scratch, size_t scratch_bytes,
                           void* stream);
/* Floating-point convolution for the network's first and last layer (fp32 weights [Cout][R][R][C] and bias on the
 * device, fp32 accumulation, zero padding, R in {1,3}, stride in {1,2}).  Two shapes are covered: few input channels
 * (C <= 16, Cout a multiple of 8, bf16 output, fp32 or bf16 input) and few output channels (Cout <= 4, C a multiple of
 * 8, bf16 input, fp32 output); anything else returns HQ_ERR_UNSUPPORTED. */
hq_status hq_conv2d_direct(const void* x, hq_dtype xdt, const float* w, const float* bias, int64_t Nb, int64_t H,
                           int64_t W, int64_t C, int64_t Cout, int R, int stride, int pad, void* y, hq_dtype ydt,
                           void* stream);
/* Self-attention core: qkv [Nb][L][3C] holds, per token, the queries of all heads, then the keys, then the values
 * (head h at columns h*dh .. of each third, dh = C / heads in {32, 48, 64, 96, 128});
 * out[n][i][h*dh ..] = sum_j softmax_j(q_i . k_j / sqrt(dh)) v_j, out [Nb][L][C].  bf16 operands on the tensor cores,
 * fp32 accumulation and softmax; the softmax weights are rounded to bf16 before they multiply the values.
 * dev_status as for the integer product (bounded waits). */
hq_status hq_attention(const void* qkv, int64_t Nb, int64_t L, int64_t C, int heads, void* out, int32_t* dev_status,
                       void* stream);

/* ---- Fused linear layer that allocates nothing and takes no workspace (the paper has no counterpart: this is a
 * packaging of hq_qlinear for a particular kind of caller, not another operation). ---------------------------------
 * Who it is for: code that must not, or cannot, obtain device memory at the moment it runs a layer -- an inference
 * loop whose memory was budgeted and handed out at start-up (a cudaMalloc there would synchronise the device and
 * could fail late), a plug-in inside a host application that owns the allocator and gives the plug-in none, or a
 * component written in a language binding that exposes kernels but not the CUDA memory API.  Such a caller still
 * owns x, the weights and y, but has nowhere to put the intermediate codes and scales that hq_qlinear keeps in its
 * `workspace` argument.  Here they live in a fixed array inside the library's device image instead:
 * HQ_NOALLOC_SCRATCH_BYTES (8 MiB) per GPU, reserved by every GPU that loads the library until the process exits.
 *
 * Same arguments, results and errors as hq_qlinear without `workspace` / `ws_bytes`, plus:
 *  - the layer must satisfy hq_workspace_size(M, K, desc->container) <= HQ_NOALLOC_SCRATCH_BYTES (for nibble codes
 *    that is M * (K/2 + 4) bytes, e.g. 8192 rows of K = 2048 is just over the limit, 8192 rows of K = 1024 fits);
 *    otherwise HQ_ERR_SCRATCH_LIMIT is returned and nothing is launched;
 *  - the first call on each device looks up the device address of the array (one CUDA runtime query, no allocation)
 *    and remembers it; make that first call with the device current and before any stream capture begins;
 *  - every call on a device uses the same array and the array keeps whatever the previous call left in it.  Nothing in
 *    it needs to start at zero (each call overwrites every byte it later reads), but two calls whose work overlaps
 *    on the GPU -- different streams, or different host threads -- race on it: keep calls on one stream, or order them
 *    with events.
 * It never calls cudaMalloc, cudaFree or any routine that allocates device or pinned memory. */
#define HQ_NOALLOC_SCRATCH_BYTES (8u * 1024u * 1024u)
hq_status hq_qlinear_noalloc(const void* x, hq_dtype xdt, int64_t M, int64_t K, int64_t ldx,
                             const hq_weight_desc* desc, const void* w_dev, const float* scale_w, const float* bias,
                             int a_bits, hq_scale_mode mode, const float* static_scale, void* y, hq_dtype ydt,
                             int64_t ldy, int32_t* dev_status, void* stream);

/* Tuning switch: where hq_qgemm, hq_qconv2d and the fused layer calls run their products on pairs of SMs
 * (tcgen05.mma.cta_group::2: each CTA of a 2-CTA cluster holds half of the weight tile or of every streamed weight block;
 * one code per byte, bf16 output, one activation scale per row or one static scale, at least 256 rows).
 *   0  nowhere;
 *   1  wherever a pair kernel covers the problem (also K_pad 128 or 384 and problems of few tiles, where it measures level
 *      or slower);
 *   2  (default) where it measured faster: reductions with streamed weights (K_pad > 512), convolutions, and two-limb
 *      weights at K_pad 512 on problems of at least one 256-row tile per SM.
 * Results are bit-identical in every mode.  Returns the previous mode.  Process-wide, not thread-safe. */
int hq_set_pair_gemm(int mode);

/* alpha of the rescale for a descriptor: 2^(-k/2) for FOLDED weights (the second normalisation of Eq. 12), else 1. */
float hq_alpha_for(const hq_weight_desc* desc);

/* ---- Measurement helper: issue-rate probe of the int8 tensor pipe (no global traffic). ---------------
 * Runs `iters` back-to-back 128x256x32 int8 MMAs per SM on resident shared-memory tiles on `ctas` CTAs.
 * The caller times it with events; ops = ctas * iters * 2*128*256*32.  dev_status as above. */
hq_status hq_mma_i8_probe(int ctas, int iters, int32_t* dev_status, void* stream);
/* The same for the paired MMA (tcgen05.mma.cta_group::2, 256x256x32 per 2-CTA cluster): `pairs` clusters;
 * ops = pairs * iters * 2*256*256*32. */
hq_status hq_mma_i8_probe_pair(int pairs, int iters, int32_t* dev_status, void* stream);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* HQ_H_ */

/*
 * flexiq.h -- C ABI of the B200 (sm_100a) FlexiQ hot path: the channel-wise mixed
 * 4/8-bit quantized GEMM and implicit-GEMM convolution with run-time low-bit ratio.
 *
 * Conventions (all entry points)
 *   - Return value: FLEXIQ_OK (0) or a negative FLEXIQ_ERR_* code.  Nothing aborts or
 *     throws across the ABI.  flexiq_last_error() returns a thread-local message for
 *     the last failing call on this thread.
 *   - "_dev" pointers are device (global) memory owned by the caller, contiguous and
 *     16-byte aligned; "_host" pointers are ordinary host memory.  The library owns
 *     only the opaque layer handles it creates, and frees them in flexiq_layer_destroy.
 *   - Device work is enqueued on the caller's stream (a cudaStream_t passed as void*,
 *     NULL = legacy default stream).  Only flexiq_layer_create_* synchronises.  The
 *     steady-state calls allocate nothing.
 *   - There is no CPU fallback: on a device that is not sm_100 the calls return
 *     FLEXIQ_ERR_UNSUPPORTED.
 *   - A layer handle belongs to the device that was current when it was created.  Every call
 *     that enqueues work for a handle returns FLEXIQ_ERR_INVALID_ARG when another device is
 *     current (its pointers would not be valid there).  One handle is used from one stream and
 *     one host thread at a time (it keeps host-side records of the calls it has enqueued);
 *     different handles may run on different streams and threads concurrently.
 *   - Every device-side wait is bounded.  If one expires the kernel raises a status
 *     word that flexiq_check_status() reports as FLEXIQ_ERR_TIMEOUT; the context
 *     stays usable.
 *
 * Notation (the paper's): K input-feature channels, split into n_g = K / G channel
 * groups of G channels; K_lo = max_4bit_ch = n_low * G channels are computed from
 * 4-bit values, the remaining K_hi = K - K_lo at 8 bits.  "Slab order" is the channel
 * order after the layout post-processing of Sec. 5: slab group j holds original group
 * group_perm[j]; channels keep their order inside a group; low-bit groups are a prefix
 * at every ratio (nested selection, Sec. 4.2).
 */
#ifndef FLEXIQ_H_
#define FLEXIQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FLEXIQ_OK 0
#define FLEXIQ_ERR_INVALID_ARG (-1)
#define FLEXIQ_ERR_UNSUPPORTED (-2)
#define FLEXIQ_ERR_CUDA (-3)
#define FLEXIQ_ERR_TIMEOUT (-4)

/* x_dtype of flexiq_quantize_lower */
#define FLEXIQ_DTYPE_F32 0
#define FLEXIQ_DTYPE_F16 1
#define FLEXIQ_DTYPE_BF16 2
#define FLEXIQ_DTYPE_I8 3 /* already quantized by Eq. 1: only lowered and gathered */

/* out_mode of flexiq_mixed_gemm / flexiq_mixed_conv */
#define FLEXIQ_OUT_ACC_I32 0    /* raw int32 accumulators                       */
#define FLEXIQ_OUT_REQUANT_I8 1 /* int8, re-quantized with y_scale (Eq. 1)      */
#define FLEXIQ_OUT_DEQUANT_F32 2 /* fp32, de-quantized                          */
/* 16-bit floating-point outputs (the evaluation runs the operators between the quantized layers,
 * normalisation and GELU, in 16-bit floating point): the DEQUANT_F32 value rounded once more, to
 * nearest even.  (3 is not a public mode.) */
#define FLEXIQ_OUT_DEQUANT_F16 4
#define FLEXIQ_OUT_DEQUANT_BF16 5

/* How the low-bit slice travels from the prologue to the mainloop (layer property).
 * PACKED : two 4-bit values per byte (half the bytes); the mainloop widens them to the
 *          tensor cores' 8-bit integer operands in shared memory.
 * MASKED : one int8 per value holding the 4-bit value already shifted back to its
 *          extraction position (x4 << sx), in ONE slab [M][K] together with the 8-bit groups
 *          (low groups first); the mainloop is a plain 8-bit integer GEMM over whole K blocks
 *          (128 channels; 64 for layers of fewer than 128): blocks below max_4bit_ch read the
 *          4-bit weights at their positions, blocks above it the 8-bit weights, and only the
 *          one block per filter tap that max_4bit_ch falls into (none when it is a multiple of
 *          the block) depends on the ratio; see flexiq_set_lowbit_ratio.
 * Both give bit-identical accumulators. */
#define FLEXIQ_LOWBIT_MASKED_I8 0
#define FLEXIQ_LOWBIT_PACKED_U4 1

typedef struct flexiq_layer *flexiq_layer_t;

/* Linear layer handle.  Implements the static part of the method: the layout
 * post-processing of Sec. 5 (input channels permuted so that same-bitwidth channels are
 * contiguous for every ratio), the per-(channel group, output channel) weight extraction
 * positions of Sec. 4.1 / Fig. 4, and the cached 4-bit weights of Sec. 7 ("Resource
 * Consumption").
 *   Wq_dev          [K][N] row-major int8, ORIGINAL channel order (8-bit model, Eq. 1)
 *   w_scale_dev     [N] fp32 per-output-channel weight scales
 *   bias_dev        [N] fp32 or NULL
 *   group_perm_host [K/G] original group stored at each slab position (a permutation)
 *   x_shift_host    [K/G] static activation extraction position (0..4) of each ORIGINAL
 *                   group (Sec. 4.1); NULL = all zero
 * K % G == 0, G in {16, 32, 64}, N % 16 == 0.  The inputs are read during the call (it
 * synchronises `stream`); they may be freed afterwards.  Starts at ratio 0. */
int flexiq_layer_create_linear(flexiq_layer_t *out, int K, int N, int group_size,
                               const int8_t *Wq_dev, const float *w_scale_dev,
                               const float *bias_dev, const int32_t *group_perm_host,
                               const uint8_t *x_shift_host, void *stream);

/* Convolution layer handle (Fig. 4): Wq_dev [Cout][R][S][Cin] int8, NHWC activations,
 * zero padding; channel groups run over Cin only, a group's extraction positions do not
 * depend on the tap.  Cin % G == 0, Cout % 16 == 0.  Otherwise as above. */
int flexiq_layer_create_conv(flexiq_layer_t *out, int Cin, int Cout, int R, int S, int stride,
                             int pad, int group_size, const int8_t *Wq_dev,
                             const float *w_scale_dev, const float *bias_dev,
                             const int32_t *group_perm_host, const uint8_t *x_shift_host,
                             void *stream);

int flexiq_layer_destroy(flexiq_layer_t layer);

/* Re-runs the layout post-processing of an existing handle for another group order (and static
 * activation positions): what flexiq_layer_create_* does with group_perm_host / x_shift_host,
 * without allocating or synchronising -- the inner loop of the selection search (Sec. 4.2), which
 * tries many selections on the same weights.  Wq_dev is the original-order weight tensor again
 * (the handle keeps only slab-order copies).  Stream-ordered after earlier calls on `stream`; the
 * ratio in force is kept.  Slabs written for the previous order no longer fit the handle. */
int flexiq_layer_set_group_perm(flexiq_layer_t layer, const int8_t *Wq_dev, const int32_t *group_perm_host,
                                const uint8_t *x_shift_host, void *stream);

/* Chooses FLEXIQ_LOWBIT_MASKED_I8 (default) or FLEXIQ_LOWBIT_PACKED_U4 for the layer.
 * Must be the same for a flexiq_quantize_lower call and the mixed_* call that consumes
 * its slabs. */
int flexiq_layer_set_lowbit_path(flexiq_layer_t layer, int lowbit_path);

/* Writes, in stream order, the one weight K block per filter tap that max_4bit_ch falls into (see
 * flexiq_set_lowbit_ratio) for the ratio in force, if the stream does not hold it already; nothing
 * on the PACKED path or when max_4bit_ch is a multiple of the block.  flexiq_quantize_lower and the
 * mixed_* calls do this themselves, also inside a stream capture, where the write always becomes
 * part of the graph: every captured graph is complete in itself, and one graph per ratio and problem
 * size can be kept and replayed in any order (Sec. 7: the ratio changes at run time without
 * re-packing the weights) with no call in between.  Kept for callers that want the write off their
 * critical path. */
int flexiq_layer_sync_ratio(flexiq_layer_t layer, void *stream);

/* Run-time ratio switch (Sec. 7, "Low-bitwidth Ratio Adjustment"): sets
 * max_4bit_ch = K_lo = ceil(ratio * n_g - 1e-4) * G, clamped to [0, K].  The call itself is
 * host-only: one integer.  Takes effect for calls enqueued afterwards.
 * What the switch costs on the device: PACKED path nothing.  MASKED path nothing when K_lo is a
 * multiple of the K block (128 channels; 64 for layers of fewer than 128 channels); otherwise the
 * next flexiq_quantize_lower (extra thread blocks of its launch) or mixed_* call (a small kernel
 * in front of it) writes the one K block per filter tap that K_lo falls into: N * taps * block
 * bytes, e.g. 393 KB for a 768 x 3072 linear layer.  The weights themselves are never re-packed.
 * The slabs a flexiq_quantize_lower call writes belong to the ratio in force when it was enqueued,
 * and the mixed_* call that reads them must be enqueued at the same ratio.  The handle remembers
 * at which max_4bit_ch it last saw each of the caller's slab buffers written (the eight most recent
 * buffers, by address: slabs of several ratios may be prepared ahead in buffers of their own), and a
 * mixed_* call that passes a remembered buffer at another ratio returns FLEXIQ_ERR_INVALID_ARG
 * instead of computing wrong values or, on the PACKED path where the row pitch depends on the ratio,
 * reading past the end of a buffer.  Buffers the handle has not seen written are taken on trust;
 * flexiq_layer_set_slab_check(layer, 0) turns the check off for callers that fill slabs themselves.
 * ratio outside [0, 1] or NaN: FLEXIQ_ERR_INVALID_ARG. */
int flexiq_set_lowbit_ratio(flexiq_layer_t layer, float ratio);
int flexiq_get_max_4bit_ch(flexiq_layer_t layer, int *K_lo);
/* enabled = 0: mixed_* calls no longer compare the ratio with the one a slab buffer was written at
 * (see flexiq_set_lowbit_ratio); any other value turns the check back on (the default). */
int flexiq_layer_set_slab_check(flexiq_layer_t layer, int enabled);

/* Row pitch in bytes of the X4_dev slab for a given K_lo under the layer's path:
 * PACKED: K_lo / 2 rounded up to a multiple of 16;  MASKED: K (the slab holds every group). */
int flexiq_x4_pitch(flexiq_layer_t layer, int K_lo, int64_t *pitch_bytes);

/* Activation prologue (Sec. 2.1 Eq. 1, Sec. 4.1 bit-lowering, Sec. 5 layout):
 *   q  = clip(round_half_even(x / x_scale), -128, 127)          (skipped for I8 input)
 *   slab group j <  n_low : x4 = clamp(q >> sx[j], -8, 7)   -> X4_dev
 *   slab group j >= n_low : q                               -> X8_dev
 * with channels gathered into slab order.
 *   X_dev    [M][K] row-major (linear) or NHWC with M = Nb*H*W pixels (conv), x_dtype
 *   X4_dev   [M][pitch] bytes, pitch = flexiq_x4_pitch(K_lo).  PACKED: byte t of a row
 *            holds slab channel 2t in bits 0-3 and 2t+1 in bits 4-7 (two's complement); may
 *            be NULL when K_lo == 0.  MASKED: the whole slab, int8 [M][K]: (x4 << sx[j]) for
 *            the low groups, then q for the 8-bit groups; never NULL.
 *   X8_dev   PACKED: [M][K_hi] int8, may be NULL when K_hi == 0.  MASKED: ignored.
 *   dynamic_pos != 0: the run-time extraction positions of Sec. 4.1 -- a bitwise OR over
 *            all values of a channel group in this call (negatives folded by ~) finds
 *            the highest used bit -- replace the static ones; they are written to
 *            x_shift_out_dev [K/G] (slab order, uint8) and must be handed to the mixed_*
 *            call.  scratch_dev must then point to K/G uint32 words of device scratch.
 * M == 0 is a successful no-op. */
int flexiq_quantize_lower(flexiq_layer_t layer, const void *X_dev, int x_dtype, int64_t M,
                          float x_scale, int dynamic_pos, uint8_t *X4_dev, int8_t *X8_dev,
                          uint8_t *x_shift_out_dev, uint32_t *scratch_dev, void *stream);

/* Dynamic-position prologue for callers that must not allocate device memory.  (The paper has
 * no counterpart; this is a convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region being captured
 * into a CUDA graph, inside a memory-pool callback or an allocator hook, in a real-time serving
 * loop that has handed all device memory to another allocator -- and that therefore cannot set
 * aside the K/G scratch words flexiq_quantize_lower(dynamic_pos = 1) asks its caller for.  This
 * entry point behaves exactly like that call (same arguments otherwise, same results), but takes
 * its scratch from a fixed array inside the library and calls no allocating routine at all.
 *
 * Limits and rules:
 *   - at most 4096 channel groups per layer (K/G <= 4096); larger layers get
 *     FLEXIQ_ERR_INVALID_ARG and should use flexiq_quantize_lower with their own scratch.
 *     The array costs 16 KB of device memory on every GPU that loads the library, until exit.
 *   - the first call on each device looks up the array's device address (with that device
 *     current) and caches it; make that first call outside any stream capture.
 *   - every call on a device shares the one array (it is cleared at the start of each call, on
 *     `stream`): calls whose kernels may overlap on the GPU -- different streams without an
 *     ordering between them -- race on it and give wrong positions.  Keep such calls ordered. */
int flexiq_quantize_lower_dynamic_noalloc(flexiq_layer_t layer, const void *X_dev, int x_dtype,
                                          int64_t M, float x_scale, uint8_t *X4_dev, int8_t *X8_dev,
                                          uint8_t *x_shift_out_dev, void *stream);

/* Mixed-precision GEMM (Sec. 7; objective of Sec. 2.3):
 *   acc[m][n] = sum_{j <  n_low} ( sum_i x4[m][j,i] * w4[j,i][n] ) << (sx[j] + sw[j][n])
 *             + sum_{j >= n_low}   sum_i x8[m][j,i] * w8[j,i][n]            (exact int32)
 * followed by the per-output-channel epilogue
 *   ACC_I32    : acc
 *   REQUANT_I8 : clip(round_half_even(fma(float(acc), (x_scale*w_scale[n])/y_scale,
 *                                        bias[n]/y_scale)), -128, 127)
 *   DEQUANT_F32: fma(float(acc), x_scale*w_scale[n], bias[n])
 *   DEQUANT_F16 / DEQUANT_BF16: that fp32 value converted to fp16 / bf16, round to nearest even
 *   X4_dev/X8_dev  slabs written by flexiq_quantize_lower at the layer's current ratio
 *   x_shift_dev    [K/G] uint8 slab-order activation positions (dynamic mode) or NULL for
 *                  the layer's static ones.  Only the PACKED path reads it; on the MASKED
 *                  path the positions are already folded into the slab.
 *   Y_dev          [M][N] row-major of the out_mode's type. */
int flexiq_mixed_gemm(flexiq_layer_t layer, const uint8_t *X4_dev, const int8_t *X8_dev,
                      const uint8_t *x_shift_dev, int64_t M, float x_scale, float y_scale,
                      int out_mode, void *Y_dev, void *stream);

/* Mixed-precision convolution as an implicit GEMM (Fig. 4): m = (image, p, q),
 * k = (r, s, c), x[image][p*stride + r - pad][q*stride + s - pad][c], zero outside; the
 * slabs are NHWC with the channel dimension laid out as in flexiq_quantize_lower
 * (X4_dev [Nb][H][W][pitch], and on the packed path X8_dev [Nb][H][W][C_hi]); Y_dev [Nb][P][Q][Cout].
 * Calls on one layer handle must be ordered on one stream (the handle's ratio-dependent weight
 * block and its epilogue factor tables follow the ratio and the scales of the calls it has seen). */
int flexiq_mixed_conv(flexiq_layer_t layer, const uint8_t *X4_dev, const int8_t *X8_dev,
                      const uint8_t *x_shift_dev, int Nb, int H, int W, float x_scale,
                      float y_scale, int out_mode, void *Y_dev, void *stream);

/* out_order of flexiq_mixed_gemm_to_slab / flexiq_mixed_conv_to_slab */
#define FLEXIQ_ORDER_ORIGINAL 0  /* output channel n of this layer is input channel n of the next one */
#define FLEXIQ_ORDER_NEXT_SLAB 1 /* this layer's output channels were permuted offline into the next layer's slab order */

/* Fused layer boundary: the mixed GEMM / convolution of `layer` whose epilogue writes the
 * activation slab of `next_layer` directly, so that no 8-bit tensor and no prologue pass lies
 * between two quantized layers.  Per output element it computes what the two-call sequence
 *   flexiq_mixed_*(..., y_scale = next_x_scale, REQUANT_I8)  [-> max(., 0) if relu]
 *   flexiq_quantize_lower(next_layer, ., FLEXIQ_DTYPE_I8, static positions)
 * computes, bit for bit: the value re-quantized by Eq. 1's rounding at the next layer's scale,
 * moved to its channel's place in the next layer's slab order (layout post-processing, Sec. 5),
 * and, when its group lies below the next layer's current max_4bit_ch, bit-lowered at the group's
 * static extraction position with saturation (Sec. 4.1) and stored as x4 << sx.
 *   next_layer     a layer on the MASKED path of the same device with K (or Cin) equal to this
 *                  layer's N (or Cout); its ratio at the time of this call decides the lowering
 *   next_x_scale   the next layer's activation scale (> 0)
 *   relu           non-zero: max(., 0) between the two layers (ResNet-style blocks)
 *   out_order      ORIGINAL: each 16-channel chunk of the result is scattered to its place in the
 *                  next layer's slab order (16-byte stores).  NEXT_SLAB: the caller created this
 *                  layer from weights, scales and biases whose output channels were already
 *                  permuted into the next layer's slab order (Sec. 5: the reordering is moved
 *                  offline into the producing layer), so channel n lands at slab channel n and
 *                  rows are written with full 32-byte stores -- the faster form.
 *   next_X4_dev    [M][N] (or [Nb][P][Q][Cout]) the next layer's slab, 16-byte aligned, caller-owned
 * Dynamic positions for the next layer are not available here (they need all rows first).
 * The paper runs the two steps as separate kernels; it has no counterpart of this fusion.
 * Errors as for flexiq_mixed_gemm, plus UNSUPPORTED when next_layer is on the PACKED path and
 * INVALID_ARG when the channel counts or devices differ. */
int flexiq_mixed_gemm_to_slab(flexiq_layer_t layer, const uint8_t *X4_dev, const int8_t *X8_dev,
                              const uint8_t *x_shift_dev, int64_t M, float x_scale,
                              flexiq_layer_t next_layer, float next_x_scale, int relu,
                              int out_order, uint8_t *next_X4_dev, void *stream);
int flexiq_mixed_conv_to_slab(flexiq_layer_t layer, const uint8_t *X4_dev, const int8_t *X8_dev,
                              const uint8_t *x_shift_dev, int Nb, int H, int W, float x_scale,
                              flexiq_layer_t next_layer, float next_x_scale, int relu,
                              int out_order, uint8_t *next_X4_dev, void *stream);

/* ---- Calibration on the device (off the hot path; produces what flexiq_layer_create_* takes) ----
 *
 * flexiq_calib_channel_ranges: per input channel the range [lo, hi] (lo <= 0 <= hi) of the
 *   Eq. 1-quantized calibration activations X_dev [M][K] (Sec. 4.2 takes the channels' ranges
 *   from a sample of calibration data).  accumulate != 0 merges into
 *   the ranges already in lo_dev / hi_dev (several calibration batches); 0 starts from [0, 0].
 *   lo_dev, hi_dev: [K] int32.  K % 16 == 0.
 * flexiq_calib_channel_histogram / flexiq_calib_ranges_from_histogram: ranges that cover a given
 *   share of each channel's values instead of all of them (Sec. 8.4 presumes ranges holding 99 % of a
 *   channel's values).  The first counts the Eq. 1-quantized values per channel,
 *   hist_dev [K][256] uint32 with bin q + 128 (accumulate as above); the second drops at most `tail`
 *   samples from each end of every channel's histogram -- the caller passes
 *   tail = floor(n * (1 - coverage) / 2) for n samples per channel -- and widens the result to
 *   contain zero.  tail = 0 gives the exact ranges of flexiq_calib_channel_ranges.
 * flexiq_calib_weight_absmax: wmax_dev[k] = max |w| over the output channels (and taps) of input
 *   channel k (Sec. 4.2 pairs an activation channel with the widest range of its weights over the
 *   output channels).  Linear: Wq_dev [K][N], taps ignored;
 *   convolution (is_conv != 0): Wq_dev [N][taps][K].
 * flexiq_calib_prepare: from those three tables, per channel group of group_size channels
 *     x_shift_dev[g]  static extraction position of ORIGINAL group g: that of its widest channel
 *                     (Sec. 4.1; used magnitude bits L -> max(0, L - 3))
 *     score_dev[g]    error-estimation score: max over the group's channels of
 *                     max(hi, -lo) * wmax (Sec. 4.2), int64
 *     perm_dev        groups by ascending score, ties by index: the greedy nested order whose
 *                     prefixes are the low-bit sets (Sec. 4.2 / Sec. 5), int32 [K/group_size]
 *     unused_hist_dev [5] number of channels with 0, 1, 2, 3, >= 4 unused magnitude bits (Sec. 8.4)
 *   perm_dev and x_shift_dev, copied to the host, are the group_perm_host / x_shift_host of
 *   flexiq_layer_create_*.
 * flexiq_calib_absmax_ema: activation range across batches by exponential moving average
 *   (Sec. 7: momentum 0.99).  state_dev: 4 floats, zeroed by the caller before the first batch;
 *   after each call state_dev[0] = momentum * previous + (1 - momentum) * max|x| of this batch
 *   (the first batch sets it to its max|x|), state_dev[1] = batches seen.  x_scale = state[0] / 127.
 *   count = number of elements, a multiple of 16; floating-point x_dtype only.
 * All enqueue on `stream`, allocate nothing and return the usual codes. */
int flexiq_calib_channel_ranges(const void *X_dev, int x_dtype, int64_t M, int K, float x_scale,
                                int accumulate, int32_t *lo_dev, int32_t *hi_dev, void *stream);
int flexiq_calib_channel_histogram(const void *X_dev, int x_dtype, int64_t M, int K, float x_scale,
                                   int accumulate, uint32_t *hist_dev, void *stream);
int flexiq_calib_ranges_from_histogram(const uint32_t *hist_dev, int K, int64_t tail, int32_t *lo_dev,
                                       int32_t *hi_dev, void *stream);
int flexiq_calib_weight_absmax(const int8_t *Wq_dev, int is_conv, int K, int N, int taps,
                               int32_t *wmax_dev, void *stream);
int flexiq_calib_prepare(const int32_t *lo_dev, const int32_t *hi_dev, const int32_t *wmax_dev, int K,
                         int group_size, int32_t *perm_dev, uint8_t *x_shift_dev, int64_t *score_dev,
                         int32_t *unused_hist_dev, void *stream);
int flexiq_calib_absmax_ema(const void *X_dev, int x_dtype, int64_t count, float momentum,
                            float *state_dev, void *stream);

/* direction of flexiq_reorder_channels */
#define FLEXIQ_REORDER_TO_SLAB 0   /* original channel order -> the layer's slab order */
#define FLEXIQ_REORDER_FROM_SLAB 1 /* the layer's slab order -> original channel order  */

/* Residual-branch reorder operator (Sec. 5, layout post-processing step 3): copies a tensor
 * while moving whole channel groups between the original channel order and the slab order of
 * `layer` (its K / Cin channels, groups of G), for tensors that travel on a residual connection
 * around layers whose outputs were permuted offline.
 *   TO_SLAB  : Y[m][j*G + i] = X[m][group_perm[j]*G + i]
 *   FROM_SLAB: Y[m][group_perm[j]*G + i] = X[m][j*G + i]
 *   X_dev, Y_dev  [M][K] elements of elem_bytes in {1, 2, 4} (int8, fp16/bf16, fp32/int32),
 *                 row-major, 16-byte aligned, distinct buffers (not in place)
 * The values are not interpreted.  M == 0 is a successful no-op. */
int flexiq_reorder_channels(flexiq_layer_t layer, const void *X_dev, int elem_bytes, int64_t M,
                            int direction, void *Y_dev, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Run-time ratio controller and request queue (Sec. 8, "Adapting to Workload Fluctuation" and
 * the Poisson serving experiment).  Host-only: no device work, no stream.
 *
 * Levels are the low-bit ratios a deployment switches between (0, 25, 50, 75, 100 % in the
 * paper: n_levels = 5, level l = ratio l / (n_levels - 1)); the caller applies a level with
 * flexiq_set_lowbit_ratio.  The controller holds the latency that was profiled per level over a
 * grid of request rates and, given the request rate it is shown, moves the level one step up
 * when the profiled latency of the current level at that rate is above the threshold; one step
 * down when the next lower level's profiled latency at that rate is within the threshold (the
 * paper states only the step up; its fluctuating-rate figure needs both).  Between two grid
 * rates the profiled latency is interpolated linearly; outside the grid the end value holds.
 *   rate_grid_host [n_rates]            requests per second, strictly ascending, n_rates >= 1
 *   latency_host   [n_levels][n_rates]  profiled latency, seconds (any statistic: median, p90)
 *   threshold      seconds;  window_s   seconds of arrivals the rate is measured over (> 0)
 * All arrays are copied; the handle is freed by flexiq_controller_destroy. */
typedef struct flexiq_controller *flexiq_controller_t;
int flexiq_controller_create(flexiq_controller_t *out, int n_levels, int n_rates, const double *rate_grid_host,
                             const double *latency_host, double threshold, double window_s, int initial_level);
int flexiq_controller_destroy(flexiq_controller_t ctrl);
int flexiq_controller_level(flexiq_controller_t ctrl, int *level);
/* one decision from an observed request rate; *level receives the level after it */
int flexiq_controller_update(flexiq_controller_t ctrl, double rate, int *level);

/* The request queue of the serving experiment in virtual time: one accelerator, first come first
 * served.  When the accelerator is free it takes every request that has arrived by then, oldest
 * first, up to max_batch (max_batch = 1: the plain single-server queue), serves the batch for
 * service_host[level][batch - 1] seconds and completes all its requests together.  With a
 * controller, a dispatch that starts at least window_s after the previous decision (the first is
 * due at time window_s) first shows the controller the rate = arrivals in the last window_s
 * before the dispatch / window_s; the controller's level is left where the run ended.  Without
 * one (ctrl NULL) every batch runs at fixed_level.
 *   arrival_host  [n]  seconds, ascending        service_host [n_levels][max_batch] seconds
 *   response_host [n]  completion - arrival      level_host   [n] level that served each request
 * n == 0 is a successful no-op.  Errors: FLEXIQ_ERR_INVALID_ARG (NULL, sizes, unsorted arrivals,
 * level out of range, n_levels different from the controller's). */
int flexiq_serving_simulate(flexiq_controller_t ctrl, int fixed_level, int64_t n, const double *arrival_host,
                            int n_levels, int max_batch, const double *service_host, double *response_host,
                            int32_t *level_host);

/* ---------------------------------------------------------------------------------------------
 * Evolutionary selection of the low-bitwidth channel groups (Sec. 4.2, Algorithm 1).
 *
 * A chromosome is one flag (uint8 0/1) per channel group, layer after layer: groups_host[l] flags
 * for layer l, `total` = their sum; 1 = computed from 4-bit values.  score_host[total] is the error
 * estimation score of each group (activation range x largest weight range, flexiq_calib_prepare's
 * score_dev; 0 <= score < 2^31).  locked_host (or NULL) marks groups that every chromosome keeps
 * set: the selection of the next smaller ratio, so that selections stay nested across ratios.
 * The fitness of a chromosome is the caller's: run the model with each layer's selected groups
 * first in group_perm and K_lo = their number, and take the squared distance of its outputs from
 * the 8-bit model's (flexiq_sq_distance_i8); smaller is fitter.
 *
 * Randomness is counter based (splitmix64 finaliser over seed, generation, individual, draw index),
 * so a run is reproducible from `seed`.  Draws that should favour low scores (Sec. 4.2) use the
 * integer weights 2^32 / (1 + score); a flag to clear is drawn with weight 1 + score.
 *
 * flexiq_evo_init: population_host [N][total] receives the seeds: chromosome 0 is the greedy
 *   selection (per layer its per_layer_target_host[l] lowest scores, ties by index, locked first),
 *   the others set the locked flags and then draw flags over the whole model, low scores preferred,
 *   until they hold as many as chromosome 0; *target_out = that number.
 * flexiq_evo_next_generation: distance_host [N] = fitness of population_host's chromosomes.  The k
 *   fittest are copied unchanged (rank order, ties by index); the other N - k places are filled pair
 *   by pair: two parents drawn among the r fittest, one crossover point at a layer boundary, the two
 *   children that swap the parts right of it (an odd last place takes the first child); then each
 *   child is mutated: every set, unlocked flag is cleared with probability mutation_bp / 10000
 *   (100 = the paper's 1 %) and as many flags of the same layer that were unset are set, low scores
 *   preferred; finally flags are cleared (high scores first in probability) or set until the
 *   chromosome holds `target` flags again.  generation >= 0 numbers the call.
 * Host-only, no device work.  Errors: FLEXIQ_ERR_INVALID_ARG. */
int flexiq_evo_init(int n_layers, const int32_t *groups_host, const int64_t *score_host,
                    const uint8_t *locked_host, const int32_t *per_layer_target_host, int N, uint64_t seed,
                    uint8_t *population_host, int64_t *target_out);
int flexiq_evo_next_generation(int n_layers, const int32_t *groups_host, const int64_t *score_host,
                               const uint8_t *locked_host, int64_t target, int N, int k, int r,
                               int mutation_bp, uint64_t seed, int generation, const int64_t *distance_host,
                               const uint8_t *population_host, uint8_t *next_population_host);

/* Fitness reduction (Sec. 4.2: L2 distance from the outputs of the high-bitwidth model), exact:
 * *out_dev = sum over i < n of (A[i] - B[i])^2 for int8 tensors, as int64.  out_dev is zeroed and
 * written in stream order; A_dev, B_dev 16-byte aligned; n == 0 gives 0. */
int flexiq_sq_distance_i8(const int8_t *A_dev, const int8_t *B_dev, int64_t n, int64_t *out_dev, void *stream);

/* Test hooks: copy the layer's derived tables to host buffers (any may be NULL).
 *   sw_host [K/G][N] uint8 weight extraction positions (slab order),
 *   w8_host [N][Kw] int8 slab-order weights, w4_host [N][Kw/2] packed 4-bit weights,
 * Kw = K (linear) or R*S*Cin with k = (r*S + s)*Cin + c (conv). */
int flexiq_layer_export(flexiq_layer_t layer, uint8_t *sw_host, int8_t *w8_host,
                        uint8_t *w4_host);

/* Test hook: forces the mainloop's tile shape for every later mixed_* call of the process
 * (cta_group 1 or 2 CTAs per tile, tile_n in {64, 128, 192, 256}; cta_group 2 needs
 * tile_n >= 128).  cta_group 0 restores the automatic choice.  The paper has no counterpart. */
int flexiq_force_tile(int cta_group, int tile_n);

/* Test hook, host-only (no GPU needed): the tile shape the automatic choice takes for a masked-path layer of
 * M rows, N output channels and k_blocks K blocks of block_k (128 or 64) bytes per tile on a GPU of sm_count
 * SMs.  Writes the CTAs per tile (1 or 2) and the tile width.  The paper has no counterpart. */
int flexiq_choose_tile(int64_t M, int N, int k_blocks, int block_k, int sm_count, int *cta_group_out, int *tile_n_out);

/* Test hook: runs the mainloop's bounded wait, with a limit of about a millisecond instead of two seconds, once on
 * a barrier that completes and once on a barrier that nothing ever arrives on.  result_dev [3] int32 receives
 * {1, 0, 1}: the first wait was served, the second gave up, and the CTA's give-up flag is set; the status word is
 * raised as after any expired wait (flexiq_check_status then returns FLEXIQ_ERR_TIMEOUT once, and the context
 * stays usable).  Nothing traps and nothing spins without bound.  The paper has no counterpart. */
int flexiq_selftest_wait_expiry(int *result_dev, void *stream);

/* Reads and clears the device status word raised by a bounded wait that expired.
 * Synchronises `stream`. */
int flexiq_check_status(void *stream);

const char *flexiq_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FLEXIQ_H_ */

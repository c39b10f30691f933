/*
 * FlexiQ CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, scalar restatement of what the mixed 4/8-bit quantized GEMM and
 * convolution of FlexiQ compute.  It shares no code, table, header or helper with the
 * CUDA library; only the tests, the smoke check and the CPU-baseline leg of the
 * benchmark may call it.  Every function names the passage of the paper it follows.
 * Loops are written in the order of the definition (per channel group: a partial dot
 * product, bit-aligned by the group's extraction positions, added to the accumulator);
 * the only concession to speed is an OpenMP "parallel for" over independent rows.
 *
 * Pinned by tests (values printed in the paper, closed forms, brute force):
 *   fqo_quantize_f32      Sec. 2.1 Eq. 1; worked examples of Sec. 4.1 (0.957 -> 29,
 *                         -0.297 -> -9).  The tie-break (round-half-even) and the use of
 *                         a true fp32 division are readings: "parity unpinned" by the paper.
 *   fqo_position_*        Sec. 4.1 examples (max < 32 -> skip 2 bits; min > -16 -> skip 3).
 *   fqo_lower             Sec. 4.1 / Fig. 3 examples (29 -> 7, -9 -> -5), bit-subset rule
 *                         of Sec. 2.3.
 *   fqo_mixed_gemm_acc    ratio 0 == int8 GEMM, ratio 1 == pure 4-bit computation,
 *                         masked-operand closed form, brute-force dot products.
 *   fqo_mixed_conv_acc    equals the GEMM on an explicit im2col matrix; ratio 0 equals a
 *                         float64 convolution of the int8 tensors.
 *   fqo_weight_*_conv     brute force over every tap per (group, output channel): no weight
 *                         saturates and one position less would; 1x1 equals the linear tables.
 *   fqo_epilogue_*        the paper gives no epilogue formula, so the FORM (which factors, in
 *                         which association) is a reading: "parity unpinned" by the paper.  The
 *                         arithmetic of that form is pinned: exact rational arithmetic on the
 *                         fp32 factors rounded once, at general scales and next to ties.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define FQO_OK 0
#define FQO_ERR_OVERFLOW (-1)
#define FQO_ERR_ARG (-2)

/* ------------------------------------------------------------------ Sec. 2.1, Eq. 1
 * x_q = clip(round(x / S), Qn, Qp) with [Qn, Qp] = [-128, 127].
 * Readings: the division is a true IEEE fp32 division as Eq. 1 writes it; the rounding
 * is to nearest, ties to even (the IEEE default rounding of nearbyintf). */
int8_t fqo_quantize_one(float x, float S)
{
    volatile float t = x / S;
    float r = nearbyintf(t);
    if (r < -128.0f) r = -128.0f;
    if (r > 127.0f) r = 127.0f;
    return (int8_t)r;
}

void fqo_quantize_f32(const float *x, int64_t n, float S, int8_t *q)
{
    for (int64_t i = 0; i < n; ++i) q[i] = fqo_quantize_one(x[i], S);
}

/* Number of bits needed to write the non-negative integer v (0 -> 0, 1 -> 1, 31 -> 5). */
int fqo_bitlen(int v)
{
    int n = 0;
    while (v > 0) { ++n; v >>= 1; }
    return n;
}

/* ------------------------------------------------------------------ Sec. 4.1
 * Extraction position of a channel whose quantized values lie in [lo, hi]: the number
 * of magnitude bits in use is L (hi < 32 uses 5, lo > -16 uses 4: the paper's two
 * examples); the 4-bit value keeps the sign plus the top three used bits, so the
 * position (right shift) is max(0, L - 3), at most 4 for 8-bit values.  Channels with
 * more than four unused bits keep position 0 (the 4-bit value is then lossless). */
int fqo_used_bits_from_range(int lo, int hi)
{
    int L = 0;
    if (hi > 0) { int b = fqo_bitlen(hi); if (b > L) L = b; }
    if (lo < 0) { int b = fqo_bitlen(~lo); if (b > L) L = b; }
    return L;
}

int fqo_position_from_range(int lo, int hi)
{
    int L = fqo_used_bits_from_range(lo, hi);
    return L > 3 ? L - 3 : 0;
}

/* Per-channel ranges of a calibration batch of quantized activations qcal[Mc][K]
 * (Sec. 4.2: ranges are estimated from sampled calibration data). */
void fqo_channel_ranges(const int8_t *qcal, int64_t Mc, int K, int32_t *lo, int32_t *hi)
{
    for (int c = 0; c < K; ++c) { lo[c] = 0; hi[c] = 0; }
    for (int64_t m = 0; m < Mc; ++m)
        for (int c = 0; c < K; ++c) {
            int v = qcal[m * K + c];
            if (v < lo[c]) lo[c] = v;
            if (v > hi[c]) hi[c] = v;
        }
}

/* Static activation position of every ORIGINAL channel group g (G consecutive channels):
 * the group's position is that of its widest channel (Sec. 7 speaks of one extraction
 * position per group). */
void fqo_static_positions(const int32_t *lo, const int32_t *hi, int K, int G, uint8_t *sx_group)
{
    for (int g = 0; g < K / G; ++g) {
        int L = 0;
        for (int i = 0; i < G; ++i) {
            int b = fqo_used_bits_from_range(lo[g * G + i], hi[g * G + i]);
            if (b > L) L = b;
        }
        sx_group[g] = (uint8_t)(L > 3 ? L - 3 : 0);
    }
}

/* ------------------------------------------------------------------ Sec. 4.2
 * Error-estimation score of a channel = activation range x the largest weight range over
 * the output channels, both in quantized units so the score is an exact integer; a
 * group's score is the largest of its channels' (reading: the paper does not say how
 * channel scores combine).  Groups sorted by ascending score, ties by index, give the
 * greedy, nested order: the low-bit set at any ratio is a prefix. Weights Wq[K][N]. */
static const int64_t *g_sort_key;
static int cmp_group(const void *a, const void *b)
{
    int32_t ia = *(const int32_t *)a, ib = *(const int32_t *)b;
    if (g_sort_key[ia] != g_sort_key[ib]) return g_sort_key[ia] < g_sort_key[ib] ? -1 : 1;
    return ia < ib ? -1 : (ia > ib);
}

void fqo_greedy_order(const int32_t *lo, const int32_t *hi, const int32_t *wabs_max /*[K]*/,
                      int K, int G, int64_t *score_group, int32_t *perm)
{
    int ng = K / G;
    for (int g = 0; g < ng; ++g) {
        int64_t best = 0;
        for (int i = 0; i < G; ++i) {
            int c = g * G + i;
            int64_t r = hi[c] > -lo[c] ? hi[c] : -lo[c];
            int64_t s = r * (int64_t)wabs_max[c];
            if (s > best) best = s;
        }
        score_group[g] = best;
        perm[g] = g;
    }
    g_sort_key = score_group;
    qsort(perm, (size_t)ng, sizeof(int32_t), cmp_group);
}

/* max_n |Wq[c][n]| for a linear weight Wq[K][N]. */
void fqo_weight_absmax_linear(const int8_t *Wq, int K, int N, int32_t *wabs_max)
{
    for (int c = 0; c < K; ++c) {
        int best = 0;
        for (int n = 0; n < N; ++n) {
            int v = Wq[(int64_t)c * N + n];
            if (v < 0) v = -v;
            if (v > best) best = v;
        }
        wabs_max[c] = best;
    }
}

/* max over output channels and taps of |Wq[n][r][s][c]| for a conv weight. */
void fqo_weight_absmax_conv(const int8_t *Wq, int Cout, int R, int S, int Cin, int32_t *wabs_max)
{
    for (int c = 0; c < Cin; ++c) wabs_max[c] = 0;
    for (int64_t i = 0; i < (int64_t)Cout * R * S; ++i)
        for (int c = 0; c < Cin; ++c) {
            int v = Wq[i * Cin + c];
            if (v < 0) v = -v;
            if (v > wabs_max[c]) wabs_max[c] = v;
        }
}

/* Number of low-bit groups for a ratio: the constraint ||beta||_0 >= target (Sec. 2.3)
 * is met by rounding up; 1e-4 absorbs the representation error of ratios like 0.75. */
int fqo_n_low(double ratio, int n_groups)
{
    int n = (int)ceil(ratio * (double)n_groups - 1e-4);
    if (n < 0) n = 0;
    if (n > n_groups) n = n_groups;
    return n;
}

/* ------------------------------------------------------------------ Sec. 4.1, Fig. 4
 * Weight extraction positions: independently per (channel group, output channel), from
 * the G weights themselves (and all taps for a conv), so weights never saturate.
 * sw is indexed [slab group j][n], slab group j being original group perm[j]. */
void fqo_weight_positions_linear(const int8_t *Wq, int K, int N, int G, const int32_t *perm,
                                 uint8_t *sw)
{
    int ng = K / G;
    for (int j = 0; j < ng; ++j)
        for (int n = 0; n < N; ++n) {
            int lo = 0, hi = 0;
            for (int i = 0; i < G; ++i) {
                int v = Wq[(int64_t)(perm[j] * G + i) * N + n];
                if (v < lo) lo = v;
                if (v > hi) hi = v;
            }
            sw[(int64_t)j * N + n] = (uint8_t)fqo_position_from_range(lo, hi);
        }
}

void fqo_weight_positions_conv(const int8_t *Wq, int Cout, int R, int S, int Cin, int G,
                               const int32_t *perm, uint8_t *sw)
{
    int ng = Cin / G;
    for (int j = 0; j < ng; ++j)
        for (int n = 0; n < Cout; ++n) {
            int lo = 0, hi = 0;
            for (int t = 0; t < R * S; ++t)
                for (int i = 0; i < G; ++i) {
                    int v = Wq[((int64_t)n * R * S + t) * Cin + perm[j] * G + i];
                    if (v < lo) lo = v;
                    if (v > hi) hi = v;
                }
            sw[(int64_t)j * Cout + n] = (uint8_t)fqo_position_from_range(lo, hi);
        }
}

/* ------------------------------------------------------------------ Sec. 4.1 (dynamic)
 * Run-time extraction position: a bitwise OR over all values of the channel group in this
 * call finds the highest bit in use.  Negative values are folded (q -> ~q) first, since
 * the OR of two's-complement negatives would always set every high bit.  One position per
 * slab group per call, over all M rows (reading). */
void fqo_dynamic_positions(const int8_t *q, int64_t M, int K, int G, const int32_t *perm,
                           uint8_t *sx_slab)
{
    int ng = K / G;
    for (int j = 0; j < ng; ++j) {
        int o = 0;
        for (int64_t m = 0; m < M; ++m)
            for (int i = 0; i < G; ++i) {
                int v = q[m * K + perm[j] * G + i];
                o |= (v >= 0) ? v : ~v;
            }
        int L = fqo_bitlen(o);
        sx_slab[j] = (uint8_t)(L > 3 ? L - 3 : 0);
    }
}

/* ------------------------------------------------------------------ Sec. 4.1, Fig. 3
 * Bit-lowering: shift the 8-bit value right by the extraction position (arithmetic
 * shift: Sec. 4.1 describes a shift followed by keeping four bits; both worked examples are floors) and keep
 * four bits.  A value outside the range the static position was chosen for saturates
 * (the paper calls such channels saturated) instead of wrapping: clamp to [-8, 7]. */
int fqo_floor_shift(int v, int s)
{
    /* floor(v / 2^s) written without relying on the sign behaviour of >> */
    return v >= 0 ? v >> s : -(((-v) + (1 << s) - 1) >> s);
}

int fqo_lower(int q, int s)
{
    int v = fqo_floor_shift(q, s);
    if (v < -8) v = -8;
    if (v > 7) v = 7;
    return v;
}

/* Canonical slabs the activation prologue must produce (for element-wise checks):
 * slab channel order = groups in perm order, channels inside a group in original order.
 * X4: row pitch x4_pitch bytes, byte t holds slab channel 2t in bits 0-3 and 2t+1 in bits
 * 4-7 as two's-complement nibbles (only the first K_lo/2 bytes of a row are written).
 * X8: [M][K_hi] the unlowered int8 values of slab groups j >= n_low. */
void fqo_make_slabs(const int8_t *q, int64_t M, int K, int G, const int32_t *perm,
                    const uint8_t *sx_slab, int n_low, uint8_t *X4, int64_t x4_pitch, int8_t *X8)
{
    int ng = K / G;
    int K_lo = n_low * G, K_hi = K - K_lo;
    for (int64_t m = 0; m < M; ++m) {
        for (int j = 0; j < n_low; ++j)
            for (int i = 0; i < G; i += 2) {
                int a = fqo_lower(q[m * K + perm[j] * G + i], sx_slab[j]);
                int b = fqo_lower(q[m * K + perm[j] * G + i + 1], sx_slab[j]);
                X4[m * x4_pitch + (j * G + i) / 2] = (uint8_t)((a & 15) | ((b & 15) << 4));
            }
        for (int j = n_low; j < ng; ++j)
            for (int i = 0; i < G; ++i)
                X8[m * K_hi + (j - n_low) * G + i] = q[m * K + perm[j] * G + i];
    }
}

/* ------------------------------------------------------------------ Sec. 7 (accumulate)
 * acc[m][n] = sum over low groups j < n_low of
 *                 ( sum_i x4[m][j,i] * w4[j,i][n] ) << (sx[j] + sw[j][n])
 *           + sum over the remaining groups of  sum_i x8[m][j,i] * w8[j,i][n]
 * x4 = lower(q, sx[j]);  w4 = Wq >> sw[j][n] (exact position, never saturates).
 * The low-bit partial sums are bit-aligned by the extraction positions and added into the
 * same accumulator as the 8-bit partial sums.  Accumulated in int64 and checked to fit
 * the int32 accumulator of the hardware.  Xq[M][K], Wq[K][N] in ORIGINAL channel order. */
int fqo_mixed_gemm_acc(const int8_t *Xq, const int8_t *Wq, int64_t M, int K, int N, int G,
                       const int32_t *perm, const uint8_t *sx_slab, const uint8_t *sw,
                       int n_low, int32_t *acc)
{
    int ng = K / G;
    int status = FQO_OK;
    if (K % G != 0 || n_low < 0 || n_low > ng) return FQO_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        int64_t *row = (int64_t *)calloc((size_t)N, sizeof(int64_t));
        int32_t *part = (int32_t *)malloc((size_t)N * sizeof(int32_t));
        for (int j = 0; j < ng; ++j) {
            int g = perm[j];
            memset(part, 0, (size_t)N * sizeof(int32_t));
            if (j < n_low) {
                for (int i = 0; i < G; ++i) {
                    int k = g * G + i;
                    int x4 = fqo_lower(Xq[m * K + k], sx_slab[j]);
                    const int8_t *wrow = Wq + (int64_t)k * N;
                    const uint8_t *s = sw + (int64_t)j * N;
                    for (int n = 0; n < N; ++n) part[n] += x4 * fqo_floor_shift(wrow[n], s[n]);
                }
                const uint8_t *s = sw + (int64_t)j * N;
                for (int n = 0; n < N; ++n)
                    row[n] += (int64_t)part[n] * ((int64_t)1 << (sx_slab[j] + s[n]));
            } else {
                for (int i = 0; i < G; ++i) {
                    int k = g * G + i;
                    int x8 = Xq[m * K + k];
                    const int8_t *wrow = Wq + (int64_t)k * N;
                    for (int n = 0; n < N; ++n) part[n] += x8 * wrow[n];
                }
                for (int n = 0; n < N; ++n) row[n] += part[n];
            }
        }
        for (int n = 0; n < N; ++n) {
            if (row[n] > INT32_MAX || row[n] < INT32_MIN) {
#pragma omp atomic write
                status = FQO_ERR_OVERFLOW;
            }
            acc[m * N + n] = (int32_t)row[n];
        }
        free(row);
        free(part);
    }
    return status;
}

/* The same accumulator for a sample of rows only (rows[i] indexes Xq); acc is [n_rows][N].
 * Used to check full-size problems on rows the oracle can afford. */
int fqo_mixed_gemm_acc_rows(const int8_t *Xq, const int8_t *Wq, const int64_t *rows,
                            int64_t n_rows, int K, int N, int G, const int32_t *perm,
                            const uint8_t *sx_slab, const uint8_t *sw, int n_low, int32_t *acc)
{
    int status = FQO_OK;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_rows; ++r) {
        int st = fqo_mixed_gemm_acc(Xq + rows[r] * K, Wq, 1, K, N, G, perm, sx_slab, sw, n_low,
                                    acc + r * N);
        if (st != FQO_OK) {
#pragma omp atomic write
            status = st;
        }
    }
    return status;
}

/* ------------------------------------------------------------------ Fig. 4 (convolution)
 * Direct convolution, NHWC activations Xq[Nb][H][W][C], weights Wq[Cout][R][S][C], zero
 * padding (the quantized zero is 0: symmetric quantization), output acc[Nb][P][Q][Cout].
 * The channel groups run over the input channels c only; a group's extraction positions do
 * not depend on the tap.  Same accumulate rule as the GEMM, one tap at a time. */
int fqo_mixed_conv_acc(const int8_t *Xq, const int8_t *Wq, int Nb, int H, int W, int C, int Cout,
                       int R, int S, int stride, int pad, int G, const int32_t *perm,
                       const uint8_t *sx_slab, const uint8_t *sw, int n_low, int32_t *acc)
{
    int ng = C / G;
    int P = (H + 2 * pad - R) / stride + 1;
    int Q = (W + 2 * pad - S) / stride + 1;
    int status = FQO_OK;
    if (C % G != 0 || n_low < 0 || n_low > ng) return FQO_ERR_ARG;
#pragma omp parallel for schedule(static) collapse(2)
    for (int b = 0; b < Nb; ++b)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int n = 0; n < Cout; ++n) {
                    int64_t sum = 0;
                    for (int r = 0; r < R; ++r)
                        for (int s = 0; s < S; ++s) {
                            int h = p * stride + r - pad, w = q * stride + s - pad;
                            if (h < 0 || h >= H || w < 0 || w >= W) continue; /* zero padding */
                            const int8_t *xpix = Xq + (((int64_t)b * H + h) * W + w) * C;
                            const int8_t *wtap = Wq + (((int64_t)n * R + r) * S + s) * C;
                            for (int j = 0; j < ng; ++j) {
                                int g = perm[j];
                                int32_t part = 0;
                                if (j < n_low) {
                                    int sh = sw[(int64_t)j * Cout + n];
                                    for (int i = 0; i < G; ++i)
                                        part += fqo_lower(xpix[g * G + i], sx_slab[j]) *
                                                fqo_floor_shift(wtap[g * G + i], sh);
                                    sum += (int64_t)part * ((int64_t)1 << (sx_slab[j] + sh));
                                } else {
                                    for (int i = 0; i < G; ++i)
                                        part += (int32_t)xpix[g * G + i] * wtap[g * G + i];
                                    sum += part;
                                }
                            }
                        }
                    if (sum > INT32_MAX || sum < INT32_MIN) {
#pragma omp atomic write
                        status = FQO_ERR_OVERFLOW;
                    }
                    acc[(((int64_t)b * P + p) * Q + q) * Cout + n] = (int32_t)sum;
                }
    return status;
}

/* ------------------------------------------------------------------ epilogue (Eq. 1 reused)
 * The paper gives no formula for the step after the accumulator beyond per-output-channel
 * scale factors (Sec. 4.1) and Eq. 1 for re-quantization; this is the standard form, every
 * operation in fp32:  alpha[n] = (S_x * S_w[n]) / S_y,  beta[n] = bias[n] / S_y,
 * y = fma(float(acc), alpha, beta) (one rounding), out = clip(round-half-even(y)). */
void fqo_epilogue_i8(const int32_t *acc, int64_t M, int N, float x_scale, const float *w_scale,
                     const float *bias, float y_scale, int8_t *out)
{
    for (int64_t m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            volatile float sxw = x_scale * w_scale[n];
            volatile float alpha = sxw / y_scale;
            volatile float beta = bias ? bias[n] / y_scale : 0.0f;
            float y = fmaf((float)acc[m * N + n], alpha, beta);
            float r = nearbyintf(y);
            if (r < -128.0f) r = -128.0f;
            if (r > 127.0f) r = 127.0f;
            out[m * N + n] = (int8_t)r;
        }
}

/* Dequantized fp32 output: y = fma(float(acc), S_x * S_w[n], bias[n]). */
void fqo_epilogue_f32(const int32_t *acc, int64_t M, int N, float x_scale, const float *w_scale,
                      const float *bias, float *out)
{
    for (int64_t m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            volatile float sxw = x_scale * w_scale[n];
            out[m * N + n] = fmaf((float)acc[m * N + n], sxw, bias ? bias[n] : 0.0f);
        }
}

/* Residual-branch reorder (Sec. 5, layout post-processing step 3): the channels of a tensor are
 * moved group by group between the original order and a layer's slab order, values untouched.
 * to_slab != 0:  y[m][j*G + i] = x[m][perm[j]*G + i];  else  y[m][perm[j]*G + i] = x[m][j*G + i].
 * Elements are elem_bytes wide and copied byte by byte. */
void fqo_reorder_channels(const uint8_t *x, int64_t M, int K, int G, int elem_bytes, const int32_t *perm,
                          int to_slab, uint8_t *y)
{
    for (int64_t m = 0; m < M; ++m)
        for (int j = 0; j < K / G; ++j)
            for (int i = 0; i < G; ++i) {
                const int64_t slab = m * K + (int64_t)j * G + i, orig = m * K + (int64_t)perm[j] * G + i;
                const int64_t dst = to_slab ? slab : orig, src = to_slab ? orig : slab;
                for (int b = 0; b < elem_bytes; ++b) y[dst * elem_bytes + b] = x[src * elem_bytes + b];
            }
}

/* Coverage-based channel ranges (Sec. 8.4 presumes ranges that hold 99 % of a channel's values): hist[c][q + 128] counts the quantized values of channel c; the range drops at most `tail`
 * samples from each end (tail = floor(n * (1 - coverage) / 2) for n samples) and is widened to contain
 * zero.  tail = 0 is the exact min / max of fqo_channel_ranges. */
void fqo_channel_histogram(const int8_t *q, int64_t M, int K, uint32_t *hist /*[K][256]*/)
{
    for (int64_t i = 0; i < (int64_t)K * 256; ++i) hist[i] = 0;
    for (int64_t m = 0; m < M; ++m)
        for (int c = 0; c < K; ++c) hist[(int64_t)c * 256 + q[m * K + c] + 128] += 1;
}
void fqo_ranges_from_histogram(const uint32_t *hist, int K, int64_t tail, int32_t *lo, int32_t *hi)
{
    for (int c = 0; c < K; ++c) {
        const uint32_t *h = hist + (int64_t)c * 256;
        int64_t dropped = 0;
        int l = -128, u = 127;
        while (l < 0 && dropped + h[l + 128] <= tail) { dropped += h[l + 128]; ++l; }
        dropped = 0;
        while (u > 0 && dropped + h[u + 128] <= tail) { dropped += h[u + 128]; --u; }
        lo[c] = l;
        hi[c] = u;
    }
}

/* Unused-bit statistics (Sec. 8.4): an int8 value has 7 magnitude bits; a channel whose range needs
 * L of them leaves 7 - L unused (Sec. 4.1's example: values below 32 leave the top two unused).  hist[u] counts the channels with u unused bits, u = 4 standing for four or more. */
void fqo_unused_bits_histogram(const int32_t *lo, const int32_t *hi, int K, int32_t *hist /*[5]*/)
{
    for (int u = 0; u < 5; ++u) hist[u] = 0;
    for (int c = 0; c < K; ++c) {
        int u = 7 - fqo_used_bits_from_range(lo[c], hi[c]);
        hist[u > 4 ? 4 : u] += 1;
    }
}

/* Activation range across batches by exponential moving average (Sec. 7, momentum 0.99): the first
 * batch sets the state to its max |x|; batch b > 0 gives state = m * state + (1 - m) * max|x_b|,
 * every operation rounded to fp32. */
float fqo_absmax_ema(const float *x, int64_t batches, int64_t per_batch, float momentum)
{
    volatile float state = 0.0f;
    for (int64_t b = 0; b < batches; ++b) {
        float a = 0.0f;
        for (int64_t i = 0; i < per_batch; ++i) {
            float v = fabsf(x[b * per_batch + i]);
            if (v > a) a = v;
        }
        if (b == 0) state = a;
        else {
            volatile float t1 = momentum * state;
            volatile float om = 1.0f - momentum;
            volatile float t2 = om * a;
            state = t1 + t2;
        }
    }
    return state;
}

int fqo_max_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

// Calibration on the device (Sec. 4.2 range estimation and error-estimation score, Sec. 7
// activation ranges by exponential moving average, Sec. 8.4 unused-bit statistics): the
// statistics that produce a layer's group order and static extraction positions, computed
// where the calibration activations already are.  Runs once per layer, off the hot path.
#include "flexiq_internal.h"

#include "sm100_ptx.cuh"
#include "eq1_quantize.cuh"

namespace flexiq {

// Loads 8 fp32 channels starting at p.
__device__ __forceinline__ void load8(const void *p, float x[8])
{
    const float4 a = __ldg(reinterpret_cast<const float4 *>(p)), b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}

// Per-channel range [lo, hi] (lo <= 0 <= hi) of the Eq. 1-quantized activations over all rows.
// A block owns a window of 256 channels (16 chunks of 16) and a slice of the rows: thread
// (chunk, row lane) walks its rows with byte-parallel min / max, the block merges in shared
// memory, then one global atomic per channel of the window.
constexpr int kCalibWindow = 256;
template <int DTYPE>
__global__ void calib_ranges_kernel(const void *__restrict__ X, long long M, int K, float S, int slices,
                                    int32_t *__restrict__ lo, int32_t *__restrict__ hi)
{
    __shared__ int lo_s[kCalibWindow], hi_s[kCalibWindow];
    lo_s[threadIdx.x] = 0;
    hi_s[threadIdx.x] = 0;
    __syncthreads();
    const int win = blockIdx.x / slices, slice = blockIdx.x - win * slices;
    const int chunk = threadIdx.x & 15, rlane = threadIdx.x >> 4;
    const int c0 = win * kCalibWindow + 16 * chunk;
    const Divider div = make_divider(S);
    if (c0 < K && DTYPE == FLEXIQ_DTYPE_I8) {
        unsigned lo_w[4] = {0, 0, 0, 0}, hi_w[4] = {0, 0, 0, 0};
        for (long long m = (long long)slice * 16 + rlane; m < M; m += (long long)slices * 16) {
            const uint4 u = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const char *>(X) + (size_t)m * K + c0));
            const unsigned w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                lo_w[k] = __vmins4(lo_w[k], w[k]);
                hi_w[k] = __vmaxs4(hi_w[k], w[k]);
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int c = 16 * chunk + 4 * k + b;
                const int l = (int)(signed char)((lo_w[k] >> (8 * b)) & 0xff), h = (int)(signed char)((hi_w[k] >> (8 * b)) & 0xff);
                if (l < 0) atomicMin(&lo_s[c], l);
                if (h > 0) atomicMax(&hi_s[c], h);
            }
    } else if (DTYPE == FLEXIQ_DTYPE_F32) {
        // Eq. 1 is monotone in x (correctly rounded division by S > 0, rounding, clipping), so the range of
        // the quantized values is the quantized range of the inputs: min / max in floating point, quantize last.
        // Eight channels per thread (32 half-chunks x 8 row lanes): sixteen running values keep the register
        // count, and with it the number of loads in flight per SM, where a bandwidth-bound kernel needs it.
        const int half = threadIdx.x & 31, rl = threadIdx.x >> 5;
        const int c8 = win * kCalibWindow + 8 * half;
        if (c8 < K) {
            float lo_f[8], hi_f[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) { lo_f[k] = 0.f; hi_f[k] = 0.f; }
            for (long long m = (long long)slice * 8 + rl; m < M; m += (long long)slices * 8) {
                float x[8];
                load8(reinterpret_cast<const char *>(X) + ((size_t)m * K + c8) * 4, x);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    lo_f[k] = fminf(lo_f[k], x[k]);
                    hi_f[k] = fmaxf(hi_f[k], x[k]);
                }
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int l = __float2int_rn(fmaxf(div(lo_f[k]), -128.f)), h = __float2int_rn(fminf(div(hi_f[k]), 127.f));
                if (l < 0) atomicMin(&lo_s[8 * half + k], l);
                if (h > 0) atomicMax(&hi_s[8 * half + k], h);
            }
        }
    } else if (c0 < K) {
        // 16-bit inputs: sixteen channels (32 bytes) per thread
        float lo_f[16], hi_f[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) { lo_f[k] = 0.f; hi_f[k] = 0.f; }
        for (long long m = (long long)slice * 16 + rlane; m < M; m += (long long)slices * 16) {
            float x[16];
            load16<DTYPE>(reinterpret_cast<const char *>(X) + ((size_t)m * K + c0) * elem_bytes<DTYPE>(), x);
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                lo_f[k] = fminf(lo_f[k], x[k]);
                hi_f[k] = fmaxf(hi_f[k], x[k]);
            }
        }
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int l = __float2int_rn(fmaxf(div(lo_f[k]), -128.f)), h = __float2int_rn(fminf(div(hi_f[k]), 127.f));
            if (l < 0) atomicMin(&lo_s[16 * chunk + k], l);
            if (h > 0) atomicMax(&hi_s[16 * chunk + k], h);
        }
    }
    __syncthreads();
    const int c = win * kCalibWindow + threadIdx.x;
    if (c < K) {
        if (lo_s[threadIdx.x] < 0) atomicMin(&lo[c], lo_s[threadIdx.x]);
        if (hi_s[threadIdx.x] > 0) atomicMax(&hi[c], hi_s[threadIdx.x]);
    }
}

// Per-channel histogram of the Eq. 1-quantized activations (256 bins, bin = q + 128), the input of
// coverage-based ranges (Sec. 8.4: ranges that cover 99 % of a channel's values).  A block owns 32
// channels and a slice of the rows and counts in shared memory; one global atomic per non-empty bin.
constexpr int kHistWindow = 32;
template <int DTYPE>
__global__ void calib_hist_kernel(const void *__restrict__ X, long long M, int K, float S, int slices, unsigned *__restrict__ hist)
{
    __shared__ unsigned h[kHistWindow * 256];
    for (int i = threadIdx.x; i < kHistWindow * 256; i += blockDim.x) h[i] = 0;
    __syncthreads();
    const int win = blockIdx.x / slices, slice = blockIdx.x - win * slices;
    const int chunk = threadIdx.x & 1, rlane = threadIdx.x >> 1;
    const int rows_per_pass = blockDim.x >> 1;
    const int c0 = win * kHistWindow + 16 * chunk;
    const Divider div = make_divider(S);
    if (c0 < K) {
        for (long long m = (long long)slice * rows_per_pass + rlane; m < M; m += (long long)slices * rows_per_pass) {
            unsigned w[4];
            quantize16<DTYPE>(reinterpret_cast<const char *>(X) + ((size_t)m * K + c0) * elem_bytes<DTYPE>(), div, -128.f, 127.f, w);
#pragma unroll
            for (int k = 0; k < 4; ++k)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const int q = (int)(signed char)((w[k] >> (8 * b)) & 0xff);
                    atomicAdd(&h[(16 * chunk + 4 * k + b) * 256 + q + 128], 1u);
                }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kHistWindow * 256; i += blockDim.x) {
        const int c = win * kHistWindow + (i >> 8);
        if (h[i] && c < K) atomicAdd(&hist[(size_t)c * 256 + (i & 255)], h[i]);
    }
}

// Range of a channel after dropping at most `tail` samples from each end of its histogram, widened to
// contain zero (lo <= 0 <= hi).  tail = 0 gives the exact min / max.
__global__ void ranges_from_hist_kernel(const unsigned *__restrict__ hist, int K, long long tail, int32_t *__restrict__ lo,
                                        int32_t *__restrict__ hi)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= K) return;
    const unsigned *h = hist + (size_t)c * 256;
    long long below = 0, above = 0;
    int l = -128, u = 127;
    while (l < 0 && below + h[l + 128] <= tail) { below += h[l + 128]; ++l; }
    while (u > 0 && above + h[u + 128] <= tail) { above += h[u + 128]; --u; }
    lo[c] = l;
    hi[c] = u;
}

// Largest |w| over the output channels (and taps) of every input channel.
// Linear weights [K][N]: one warp per input channel (row).
__global__ void weight_absmax_rows_kernel(const int8_t *__restrict__ W, int K, int N, int32_t *__restrict__ wmax)
{
    const int row = (int)(((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (row >= K) return;
    const int8_t *w = W + (size_t)row * N;
    int best = 0;
    for (int n = lane; n < N; n += 32) best = max(best, abs((int)w[n]));
    best = __reduce_max_sync(0xffffffffu, best);
    if (lane == 0) wmax[row] = best;
}
// Convolution weights [rows = Cout*R*S][Cin]: a thread per input channel, rows split over blockIdx.y.
__global__ void weight_absmax_cols_kernel(const int8_t *__restrict__ W, long long rows, int C, int32_t *__restrict__ wmax)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    int best = 0;
    for (long long r = blockIdx.y; r < rows; r += gridDim.y) best = max(best, abs((int)W[(size_t)r * C + c]));
    if (best > 0) atomicMax(&wmax[c], best);
}

__device__ __forceinline__ int used_bits(int lo, int hi)  // magnitude bits a range [lo, hi] needs (Sec. 4.1)
{
    int L = 0;
    if (hi > 0) L = 32 - __clz(hi);
    if (lo < 0) L = max(L, 32 - __clz(~lo));
    return L;
}

// From channel ranges and weight ranges: the static extraction position of every channel group
// (position of its widest channel), the group's error-estimation score (largest activation range x
// largest weight range over its channels, Sec. 4.2), the greedy order (ascending score, ties by
// index; rank counting, one block) and the histogram of channels by unused magnitude bits (0..4+).
__global__ void calib_prepare_kernel(const int32_t *__restrict__ lo, const int32_t *__restrict__ hi,
                                     const int32_t *__restrict__ wmax, int K, int G, int32_t *__restrict__ perm,
                                     uint8_t *__restrict__ x_shift, long long *score, int32_t *__restrict__ hist)
{
    __shared__ int hist_s[5];
    const int n_g = K / G;
    if (threadIdx.x < 5) hist_s[threadIdx.x] = 0;
    __syncthreads();
    for (int g = threadIdx.x; g < n_g; g += blockDim.x) {
        int L = 0;
        long long best = 0;
        for (int i = 0; i < G; ++i) {
            const int c = g * G + i;
            L = max(L, used_bits(lo[c], hi[c]));
            const long long r = max(hi[c], -lo[c]);
            best = max(best, r * (long long)wmax[c]);
        }
        x_shift[g] = (uint8_t)(L > 3 ? L - 3 : 0);
        score[g] = best;
    }
    for (int c = threadIdx.x; c < K; c += blockDim.x) atomicAdd(&hist_s[min(4, 7 - used_bits(lo[c], hi[c]))], 1);
    __syncthreads();  // the scores are complete (global writes of this block are visible to it after the barrier)
    for (int g = threadIdx.x; g < n_g; g += blockDim.x) {
        const long long s = score[g];
        int rank = 0;
        for (int o = 0; o < n_g; ++o) {
            const long long so = score[o];
            rank += (so < s) || (so == s && o < g);
        }
        perm[rank] = g;
    }
    if (threadIdx.x < 5) hist[threadIdx.x] = hist_s[threadIdx.x];
}

// Activation range by exponential moving average (Sec. 7): absmax of the batch, then
// state[0] <- momentum * state[0] + (1 - momentum) * absmax (the first batch initialises it).
// state = { ema, batches seen, scratch (absmax bits), unused }.
template <int DTYPE>
__global__ void absmax_kernel(const void *__restrict__ X, long long count, float *__restrict__ state)
{
    float best = 0.f;
    const long long n16 = count / 16;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (long long)gridDim.x * blockDim.x) {
        float x[16];
        load16<DTYPE>(reinterpret_cast<const char *>(X) + (size_t)i * 16 * elem_bytes<DTYPE>(), x);
#pragma unroll
        for (int k = 0; k < 16; ++k) best = fmaxf(best, fabsf(x[k]));
    }
    best = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(best)));  // non-negative floats order as their bits
    if ((threadIdx.x & 31) == 0 && best > 0.f) atomicMax(reinterpret_cast<unsigned *>(state + 2), __float_as_uint(best));
}
__global__ void ema_update_kernel(float *state, float momentum)
{
    const float a = state[2];
    if (state[1] == 0.f) state[0] = a;
    else state[0] = __fadd_rn(__fmul_rn(momentum, state[0]), __fmul_rn(__fsub_rn(1.f, momentum), a));
    state[1] += 1.f;
    state[2] = 0.f;
}

template <int DTYPE>
static int launch_ranges(const void *X, long long M, int K, float S, int32_t *lo, int32_t *hi, int sms, cudaStream_t st)
{
    const int windows = (K + kCalibWindow - 1) / kCalibWindow;
    long long slices = ((long long)sms * 3 + windows - 1) / windows;   // about three blocks per SM: few, long-lived blocks amortise the merge
    const long long max_slices = (M + 15) / 16;   // (fewer rows than lanes leave lanes idle, nothing more)
    if (slices > max_slices) slices = max_slices;
    calib_ranges_kernel<DTYPE><<<(unsigned)(windows * slices), kCalibWindow, 0, st>>>(X, M, K, S, (int)slices, lo, hi);
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    return FLEXIQ_OK;
}

}  // namespace flexiq

using namespace flexiq;

extern "C" int flexiq_calib_channel_ranges(const void *X_dev, int x_dtype, int64_t M, int K, float x_scale, int accumulate,
                                           int32_t *lo_dev, int32_t *hi_dev, void *stream)
{
    if (M < 0 || K <= 0 || K % 16 != 0)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "bad shape M=%lld K=%d (K must be a positive multiple of 16)", (long long)M, K);
    if (x_dtype < FLEXIQ_DTYPE_F32 || x_dtype > FLEXIQ_DTYPE_I8) return set_error(FLEXIQ_ERR_INVALID_ARG, "unknown x_dtype %d", x_dtype);
    if (x_dtype != FLEXIQ_DTYPE_I8 && !(x_scale > 0.0f)) return set_error(FLEXIQ_ERR_INVALID_ARG, "x_scale %g must be positive", (double)x_scale);
    if (!lo_dev || !hi_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "lo_dev or hi_dev is NULL");
    int rc = check_device_sm100();
    if (rc) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (!accumulate) {
        FLEXIQ_CUDA_TRY(cudaMemsetAsync(lo_dev, 0, sizeof(int32_t) * K, st));
        FLEXIQ_CUDA_TRY(cudaMemsetAsync(hi_dev, 0, sizeof(int32_t) * K, st));
    }
    if (M == 0) return FLEXIQ_OK;
    if (!X_dev || (reinterpret_cast<uintptr_t>(X_dev) & 15)) return set_error(FLEXIQ_ERR_INVALID_ARG, "X_dev is NULL or not 16-byte aligned");
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    switch (x_dtype) {
        case FLEXIQ_DTYPE_F32: return launch_ranges<FLEXIQ_DTYPE_F32>(X_dev, M, K, x_scale, lo_dev, hi_dev, sms, st);
        case FLEXIQ_DTYPE_F16: return launch_ranges<FLEXIQ_DTYPE_F16>(X_dev, M, K, x_scale, lo_dev, hi_dev, sms, st);
        case FLEXIQ_DTYPE_BF16: return launch_ranges<FLEXIQ_DTYPE_BF16>(X_dev, M, K, x_scale, lo_dev, hi_dev, sms, st);
        default: return launch_ranges<FLEXIQ_DTYPE_I8>(X_dev, M, K, x_scale, lo_dev, hi_dev, sms, st);
    }
}

extern "C" int flexiq_calib_channel_histogram(const void *X_dev, int x_dtype, int64_t M, int K, float x_scale, int accumulate,
                                              uint32_t *hist_dev, void *stream)
{
    if (M < 0 || K <= 0 || K % 16 != 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "bad shape M=%lld K=%d (K must be a positive multiple of 16)", (long long)M, K);
    if (x_dtype < FLEXIQ_DTYPE_F32 || x_dtype > FLEXIQ_DTYPE_I8) return set_error(FLEXIQ_ERR_INVALID_ARG, "unknown x_dtype %d", x_dtype);
    if (x_dtype != FLEXIQ_DTYPE_I8 && !(x_scale > 0.0f)) return set_error(FLEXIQ_ERR_INVALID_ARG, "x_scale %g must be positive", (double)x_scale);
    if (!hist_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "hist_dev is NULL");
    int rc = check_device_sm100();
    if (rc) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (!accumulate) FLEXIQ_CUDA_TRY(cudaMemsetAsync(hist_dev, 0, sizeof(uint32_t) * 256 * (size_t)K, st));
    if (M == 0) return FLEXIQ_OK;
    if (!X_dev || (reinterpret_cast<uintptr_t>(X_dev) & 15)) return set_error(FLEXIQ_ERR_INVALID_ARG, "X_dev is NULL or not 16-byte aligned");
    int dev = 0;
    cudaGetDevice(&dev);
    const int sms = device_sm_count(dev);
    const int windows = (K + kHistWindow - 1) / kHistWindow;
    long long slices = ((long long)sms * 4 + windows - 1) / windows;
    const long long max_slices = (M + 127) / 128;
    if (slices > max_slices) slices = max_slices;
    const unsigned grid = (unsigned)(windows * slices);
    switch (x_dtype) {
        case FLEXIQ_DTYPE_F32: calib_hist_kernel<FLEXIQ_DTYPE_F32><<<grid, 256, 0, st>>>(X_dev, M, K, x_scale, (int)slices, hist_dev); break;
        case FLEXIQ_DTYPE_F16: calib_hist_kernel<FLEXIQ_DTYPE_F16><<<grid, 256, 0, st>>>(X_dev, M, K, x_scale, (int)slices, hist_dev); break;
        case FLEXIQ_DTYPE_BF16: calib_hist_kernel<FLEXIQ_DTYPE_BF16><<<grid, 256, 0, st>>>(X_dev, M, K, x_scale, (int)slices, hist_dev); break;
        default: calib_hist_kernel<FLEXIQ_DTYPE_I8><<<grid, 256, 0, st>>>(X_dev, M, K, x_scale, (int)slices, hist_dev); break;
    }
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    return FLEXIQ_OK;
}

extern "C" int flexiq_calib_ranges_from_histogram(const uint32_t *hist_dev, int K, int64_t tail, int32_t *lo_dev, int32_t *hi_dev,
                                                  void *stream)
{
    if (K <= 0 || tail < 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "bad K = %d or tail = %lld", K, (long long)tail);
    if (!hist_dev || !lo_dev || !hi_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "a device pointer is NULL");
    int rc = check_device_sm100();
    if (rc) return rc;
    ranges_from_hist_kernel<<<(K + 127) / 128, 128, 0, reinterpret_cast<cudaStream_t>(stream)>>>(hist_dev, K, (long long)tail, lo_dev, hi_dev);
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    return FLEXIQ_OK;
}

extern "C" int flexiq_calib_weight_absmax(const int8_t *Wq_dev, int is_conv, int K, int N, int taps, int32_t *wmax_dev, void *stream)
{
    if (K <= 0 || N <= 0 || (is_conv && taps <= 0)) return set_error(FLEXIQ_ERR_INVALID_ARG, "bad shape K=%d N=%d taps=%d", K, N, taps);
    if (!Wq_dev || !wmax_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "Wq_dev or wmax_dev is NULL");
    int rc = check_device_sm100();
    if (rc) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (!is_conv) {
        const long long threads = (long long)K * 32;
        weight_absmax_rows_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(Wq_dev, K, N, wmax_dev);
    } else {
        FLEXIQ_CUDA_TRY(cudaMemsetAsync(wmax_dev, 0, sizeof(int32_t) * K, st));
        const long long rows = (long long)N * taps;
        const unsigned gy = (unsigned)(rows < 64 ? rows : 64);
        weight_absmax_cols_kernel<<<dim3((K + 127) / 128, gy), 128, 0, st>>>(Wq_dev, rows, K, wmax_dev);
    }
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    return FLEXIQ_OK;
}

extern "C" int flexiq_calib_prepare(const int32_t *lo_dev, const int32_t *hi_dev, const int32_t *wmax_dev, int K, int group_size,
                                    int32_t *perm_dev, uint8_t *x_shift_dev, int64_t *score_dev, int32_t *unused_hist_dev,
                                    void *stream)
{
    if (group_size != 16 && group_size != 32 && group_size != 64)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "group_size %d is not one of 16, 32, 64", group_size);
    if (K <= 0 || K % group_size != 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "K = %d is not a positive multiple of the group size", K);
    if (!lo_dev || !hi_dev || !wmax_dev || !perm_dev || !x_shift_dev || !score_dev || !unused_hist_dev)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "a device pointer is NULL");
    int rc = check_device_sm100();
    if (rc) return rc;
    calib_prepare_kernel<<<1, 1024, 0, reinterpret_cast<cudaStream_t>(stream)>>>(lo_dev, hi_dev, wmax_dev, K, group_size, perm_dev, x_shift_dev,
                                                                                 reinterpret_cast<long long *>(score_dev), unused_hist_dev);
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    return FLEXIQ_OK;
}

extern "C" int flexiq_calib_absmax_ema(const void *X_dev, int x_dtype, int64_t count, float momentum, float *state_dev, void *stream)
{
    if (count < 0 || count % 16 != 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "count = %lld must be a non-negative multiple of 16", (long long)count);
    if (x_dtype < FLEXIQ_DTYPE_F32 || x_dtype > FLEXIQ_DTYPE_BF16) return set_error(FLEXIQ_ERR_INVALID_ARG, "x_dtype %d is not a floating-point type", x_dtype);
    if (!(momentum >= 0.0f && momentum <= 1.0f)) return set_error(FLEXIQ_ERR_INVALID_ARG, "momentum %g outside [0, 1]", (double)momentum);
    if (!state_dev || (count > 0 && (!X_dev || (reinterpret_cast<uintptr_t>(X_dev) & 15))))
        return set_error(FLEXIQ_ERR_INVALID_ARG, "state_dev / X_dev is NULL or X_dev is not 16-byte aligned");
    int rc = check_device_sm100();
    if (rc) return rc;
    if (count == 0) return FLEXIQ_OK;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    long long blocks = (count / 16 + 255) / 256;
    if (blocks > (long long)sms * 8) blocks = (long long)sms * 8;
    if (x_dtype == FLEXIQ_DTYPE_F32) absmax_kernel<FLEXIQ_DTYPE_F32><<<(unsigned)blocks, 256, 0, st>>>(X_dev, count, state_dev);
    else if (x_dtype == FLEXIQ_DTYPE_F16) absmax_kernel<FLEXIQ_DTYPE_F16><<<(unsigned)blocks, 256, 0, st>>>(X_dev, count, state_dev);
    else absmax_kernel<FLEXIQ_DTYPE_BF16><<<(unsigned)blocks, 256, 0, st>>>(X_dev, count, state_dev);
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    ema_update_kernel<<<1, 1, 0, st>>>(state_dev, momentum);
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    return FLEXIQ_OK;
}

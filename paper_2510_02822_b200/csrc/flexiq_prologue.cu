// Activation prologue: quantize (Sec. 2.1, Eq. 1), bit-lower (Sec. 4.1, Fig. 3) and
// gather the channel groups into slab order (Sec. 5), writing the low-bit slab and the
// 8-bit slab that the mainloop consumes.  One pass over X (two in the dynamic
// extraction-position mode), 128-bit loads and stores, one 16-channel chunk per thread.
#include "flexiq_internal.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "sm100_ptx.cuh"
#include "eq1_quantize.cuh"
#include "straddle.cuh"

#include <stdlib.h>

namespace flexiq {

__device__ __forceinline__ int position_from_or(unsigned o)
{
    const int used = 32 - __clz(o);  // highest bit in use among the folded values
    return used > 3 ? used - 3 : 0;
}

// Phase 1 of the dynamic mode (Sec. 4.1): OR of the sign-folded quantized values of each
// slab group over all rows.  A thread keeps one chunk column and walks rows; lanes that
// hold the same group merge with a warp reduction, then one shared and one global atomic.
template <int DTYPE>
__global__ void group_or_kernel(const void *__restrict__ X, long long M, int K, int G, float S,
                                const int32_t *__restrict__ perm, unsigned *__restrict__ or_words)
{
    extern __shared__ unsigned or_s[];
    const int n_c16 = K / 16, c_per_g = G / 16, n_g = K / G;
    for (int i = threadIdx.x; i < n_g; i += blockDim.x) or_s[i] = 0;
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();  // the kernel before this one in the stream may still be producing X
    __syncthreads();
    // grid-wide thread count is a multiple of n_c16, so each thread keeps its chunk column
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    const long long rows_per_pass = nthreads / n_c16;
    const int c16 = (int)(tid % n_c16);
    const int j = c16 / c_per_g;
    const Divider div = make_divider(S);
    unsigned o = 0;
    if (tid < rows_per_pass * n_c16) {
        const int src_c = perm[j] * G + (c16 % c_per_g) * 16;
        for (long long m = tid / n_c16; m < M; m += rows_per_pass) {
            unsigned w[4];
            quantize16<DTYPE>(reinterpret_cast<const char *>(X) + ((size_t)m * K + src_c) * elem_bytes<DTYPE>(), div, -128.f, 127.f, w);
            // fold negatives per byte (q >= 0 ? q : ~q): xor with the byte's sign replicated
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned sign = (w[k] >> 7) & 0x01010101u;
                o |= w[k] ^ (sign * 0xffu);
            }
        }
    }
    o = (o | (o >> 8) | (o >> 16) | (o >> 24)) & 0xffu;  // OR of the four byte lanes
    const unsigned peers = __match_any_sync(0xffffffffu, j);
    const unsigned merged = __reduce_or_sync(peers, o);
    if ((threadIdx.x & 31) == (__ffs(peers) - 1) && merged) atomicOr(&or_s[j], merged);
    __syncthreads();
    for (int i = threadIdx.x; i < n_g; i += blockDim.x)
        if (or_s[i]) atomicOr(&or_words[i], or_s[i]);
}

// Phase 2 of the dynamic mode on the masked path: the low groups of the slab that phase 1 wrote are lowered in
// place with the positions the OR words give -- clip to what four bits hold at the position, clear the bits below
// it -- 16 bytes per thread; a group whose position is 0 is already what it should be and is not touched.  The
// positions go to sx_out (slab order).  Blocks in front: the straddle block of the weights, as in the static kernel.
__global__ void lower_inplace_kernel(int8_t *__restrict__ slab, long long M, int K, int G, int K_lo,
                                     const unsigned *__restrict__ or_words, uint8_t *__restrict__ sx_out, StraddleJob wp)
{
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();  // phase 1 has written the slab and the OR words
    if (blockIdx.x < wp.first_block) {
        const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
        if (idx < (long long)wp.rows * (wp.BK >> 4)) straddle_write_unit(wp, idx);
        return;
    }
    const unsigned qblock = blockIdx.x - wp.first_block, qblocks = gridDim.x - wp.first_block;
    if (qblock == 0)
        for (int j = threadIdx.x; j < K / G; j += blockDim.x) sx_out[j] = (uint8_t)position_from_or(or_words[j]);
    const int lo_c16 = K_lo / 16, c_per_g = G / 16;
    const long long total = M * lo_c16;
    for (long long idx = (long long)qblock * blockDim.x + threadIdx.x; idx < total; idx += (long long)qblocks * blockDim.x) {
        const long long m = idx / lo_c16;
        const int c16 = (int)(idx - m * lo_c16);
        const int s = position_from_or(or_words[c16 / c_per_g]);
        if (s == 0) continue;
        uint4 *ptr = reinterpret_cast<uint4 *>(slab + (size_t)m * K + (size_t)c16 * 16);
        const uint4 u = *ptr;
        const unsigned in[4] = {u.x, u.y, u.z, u.w};
        unsigned w[4];
        const int hi = (8 << s) - 1, lo = -(8 << s);
        const unsigned mask = ((0xffu << s) & 0xffu) * 0x01010101u;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            int b[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) b[t] = max(lo, min(hi, (int)(signed char)((in[k] >> (8 * t)) & 0xff)));
            w[k] = pack2_sat_s8(b[1], b[0], pack2_sat_s8(b[3], b[2], 0u)) & mask;
        }
        *ptr = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// Quantize + lower + gather.  Thread <-> (row m, 16-channel slab chunk c16).
//   sx != nullptr : static positions (slab order);  else positions from or_words.
// Lowering works on the packed int8 words: q is first clipped to the range the 4-bit value
// at position s can hold, [-2^(s+3), 2^(s+3) - 1] (identical to clamping q >> s to [-8, 7],
// the shift being monotone); then bits s..s+3 of every byte are the two's-complement nibble
// (packed path), and clearing the s low bits of every byte is (q >> s) << s (masked path).
// PACKED == 2 is phase 1 of the dynamic mode on the masked path: nothing is lowered yet (every group is written
// at 8 bits, gathered into slab order) and the OR of the sign-folded values of every group is collected on the way
// (or_acc; a thread keeps its chunk column from one grid stride to the next when the stride is a multiple of the
// row's chunks, which the launch arranges, so it flushes its OR once), so that the input is read once.
template <int DTYPE, int PACKED>
__global__ void quantize_lower_kernel(const void *__restrict__ X, long long M, int K, int G, int K_lo, float S,
                                      const int32_t *__restrict__ perm, const uint8_t *__restrict__ sx,
                                      const unsigned *__restrict__ or_words, uint8_t *__restrict__ X4,
                                      long long x4_pitch, int8_t *__restrict__ X8, long long x8_pitch, uint8_t *__restrict__ sx_out,
                                      StraddleJob wp)
{
    const int n_c16 = K / 16, c_per_g = G / 16, lo_c16 = K_lo / 16;
    const long long total = M * n_c16;
    const Divider div = make_divider(S);
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();  // the previous kernel may still read the slabs this one overwrites, or write X
    if (blockIdx.x < wp.first_block) {
        // Extra blocks in front of the quantizing ones (so that they run beside the first wave, not behind the
        // last): the weight K block that max_4bit_ch falls into, for the GEMM that consumes these slabs -- the
        // only weight data that depends on the ratio -- 16 bytes per thread.
        const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
        if (idx < (long long)wp.rows * (wp.BK >> 4)) straddle_write_unit(wp, idx);
        return;
    }
    const unsigned qblock = blockIdx.x - wp.first_block, qblocks = gridDim.x - wp.first_block;
    if (PACKED == 2) {
        extern __shared__ unsigned or_s[];
        unsigned *or_acc = const_cast<unsigned *>(or_words);
        const int n_g = K / G;
        for (int i = threadIdx.x; i < n_g; i += blockDim.x) or_s[i] = 0;
        __syncthreads();
        unsigned o = 0;
        int oj = -1;
        for (long long idx = (long long)qblock * blockDim.x + threadIdx.x; idx < total; idx += (long long)qblocks * blockDim.x) {
            const long long m = idx / n_c16;
            const int c16 = (int)(idx - m * n_c16);
            const int j = c16 / c_per_g;
            if (j != oj) {   // another group (only when the stride is not a multiple of a row's chunks)
                if (o) atomicOr(&or_s[oj], (o | (o >> 8) | (o >> 16) | (o >> 24)) & 0xffu);
                o = 0;
                oj = j;
            }
            const int src_c = perm[j] * G + (c16 % c_per_g) * 16;
            unsigned w[4];
            quantize16<DTYPE>(reinterpret_cast<const char *>(X) + ((size_t)m * K + src_c) * elem_bytes<DTYPE>(), div, -128.f, 127.f, w);
            *reinterpret_cast<uint4 *>(X4 + m * x4_pitch + (size_t)c16 * 16) = make_uint4(w[0], w[1], w[2], w[3]);
#pragma unroll
            for (int k = 0; k < 4; ++k) {   // fold negatives per byte (q >= 0 ? q : ~q): xor with the byte's sign replicated
                const unsigned sign = (w[k] >> 7) & 0x01010101u;
                o |= w[k] ^ (sign * 0xffu);
            }
        }
        if (o) atomicOr(&or_s[oj], (o | (o >> 8) | (o >> 16) | (o >> 24)) & 0xffu);
        __syncthreads();
        for (int i = threadIdx.x; i < n_g; i += blockDim.x)
            if (or_s[i]) atomicOr(&or_acc[i], or_s[i]);
        return;
    }
    if (sx_out != nullptr && qblock == 0)
        for (int j = threadIdx.x; j < K / G; j += blockDim.x) sx_out[j] = (uint8_t)position_from_or(or_words[j]);
    for (long long idx = (long long)qblock * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)qblocks * blockDim.x) {
        const long long m = idx / n_c16;
        const int c16 = (int)(idx - m * n_c16);
        const int j = c16 / c_per_g;
        const int src_c = perm[j] * G + (c16 % c_per_g) * 16;
        const void *src = reinterpret_cast<const char *>(X) + ((size_t)m * K + src_c) * elem_bytes<DTYPE>();
        unsigned w[4];
        if (!PACKED) {
            // Masked path: one instruction stream for both kinds of group (a warp spans the boundary in most rows).
            // A low group keeps bits s..s+3 of values clipped to what four bits hold at position s; an 8-bit group
            // is the same with the full range and nothing cleared.  The slab is [M][K]: X8 is X4 + K_lo.
            const bool low = c16 < lo_c16;
            const int s = low ? (sx ? (int)sx[j] : position_from_or(or_words[j])) : 4;
            const float bound = (float)(8 << s);
            quantize16<DTYPE>(src, div, -bound, bound - 1.f, w);
            const unsigned mask = low ? ((0xffu << s) & 0xffu) * 0x01010101u : 0xffffffffu;
            *reinterpret_cast<uint4 *>(X4 + m * x4_pitch + (size_t)c16 * 16) =
                make_uint4(w[0] & mask, w[1] & mask, w[2] & mask, w[3] & mask);
        } else if (c16 < lo_c16) {
            const int s = sx ? (int)sx[j] : position_from_or(or_words[j]);
            const float bound = (float)(8 << s);
            quantize16<DTYPE>(src, div, -bound, bound - 1.f, w);
            if (PACKED) {
                unsigned h[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const unsigned n = (w[k] >> s) & 0x0f0f0f0fu;  // one nibble per byte
                    h[k] = n | (n >> 4);                            // bytes 0 and 2 now hold two nibbles each
                }
                *reinterpret_cast<uint2 *>(X4 + m * x4_pitch + (size_t)c16 * 8) =
                    make_uint2(__byte_perm(h[0], h[1], 0x6420), __byte_perm(h[2], h[3], 0x6420));
            } else {
                const unsigned keep = (0xffu << s) & 0xffu;
                const unsigned mask = keep * 0x01010101u;
                *reinterpret_cast<uint4 *>(X4 + m * x4_pitch + (size_t)c16 * 16) =
                    make_uint4(w[0] & mask, w[1] & mask, w[2] & mask, w[3] & mask);
            }
        } else {
            quantize16<DTYPE>(src, div, -128.f, 127.f, w);
            *reinterpret_cast<uint4 *>(X8 + m * x8_pitch + (size_t)(c16 - lo_c16) * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

// Scratch of the allocation-free dynamic prologue: one OR word per channel group.  The array
// lives in the library image, so every GPU that loads the library holds these 16 KB until the
// process exits.  All calls on a device share it.
constexpr int kStaticScratchGroups = 4096;
static __device__ __align__(256) unsigned g_static_group_or[kStaticScratchGroups];

// Device address of the array above on the current device.  In host code the array's name is
// only a handle for the runtime, not a device pointer, so the address is looked up with
// cudaGetSymbolAddress -- once per device, with that device current -- and cached.
static int static_scratch_address(unsigned **out)
{
    static unsigned *cached[64] = {};
    int dev = 0;
    FLEXIQ_CUDA_TRY(cudaGetDevice(&dev));   // the caller has checked that this is the layer's device
    if (dev < 0 || dev >= 64) return set_error(FLEXIQ_ERR_UNSUPPORTED, "device ordinal %d is beyond the 64 this entry point tracks", dev);
    if (cached[dev] == nullptr) {
        void *p = nullptr;
        FLEXIQ_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_group_or));
        if (p == nullptr) return set_error(FLEXIQ_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        cached[dev] = static_cast<unsigned *>(p);
    }
    *out = cached[dev];
    return FLEXIQ_OK;
}

// Launch with programmatic stream serialization allowed (see pdl_wait in the kernels).
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned blocks, unsigned threads, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks, 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <int DTYPE>
static int launch_prologue(Layer *L, const void *X, long long M, float S, int dynamic, uint8_t *X4,
                           long long pitch, int8_t *X8, long long pitch8, uint8_t *sx_out, unsigned *scratch, cudaStream_t st)
{
    const int K = L->C, G = L->G;
    const int n_c16 = K / 16;
    const int sms = device_sm_count(L->device);
    const int threads = 256;
    const bool masked = L->lowbit_path == FLEXIQ_LOWBIT_MASKED_I8;
    if (dynamic && masked) {
        // the input is read once: phase 1 quantizes, gathers and collects the OR words, phase 2 lowers the low groups of
        // the slab in place (from L2) with the positions those words give
        FLEXIQ_CUDA_TRY(cudaMemsetAsync(scratch, 0, sizeof(unsigned) * L->n_g, st));
        long long want1 = (M * n_c16 + threads - 1) / threads;
        long long blocks1 = want1 < (long long)sms * 16 ? want1 : (long long)sms * 16;
        // a grid stride that is a multiple of a row's chunks keeps every thread on its chunk column
        int a = n_c16, b = threads;
        while (b) { const int t = a % b; a = b; b = t; }
        const long long unit = n_c16 / a;
        if (blocks1 >= unit) blocks1 -= blocks1 % unit;
        StraddleJob none{};
        FLEXIQ_CUDA_TRY(launch_pdl(quantize_lower_kernel<DTYPE, 2>, (unsigned)blocks1, threads, sizeof(unsigned) * L->n_g, st, X, M, K, G, 0, S, L->perm,
                                   static_cast<const uint8_t *>(nullptr), static_cast<const unsigned *>(scratch), X4, pitch, X8, pitch8,
                                   static_cast<uint8_t *>(nullptr), none));
    } else
    if (dynamic) {
        FLEXIQ_CUDA_TRY(cudaMemsetAsync(scratch, 0, sizeof(unsigned) * L->n_g, st));
        long long want = (M * n_c16 + threads - 1) / threads;
        long long blocks = want < (long long)sms * 8 ? want : (long long)sms * 8;
        // thread count must cover at least one full row of chunks
        while (blocks * threads < n_c16) ++blocks;
        FLEXIQ_CUDA_TRY(launch_pdl(group_or_kernel<DTYPE>, (unsigned)blocks, threads, sizeof(unsigned) * L->n_g, st, X, M, K, G, S, L->perm, scratch));
    }
    long long want = (M * n_c16 + threads - 1) / threads;
    long long blocks = want < (long long)sms * 16 ? want : (long long)sms * 16;
    const uint8_t *sx = dynamic ? nullptr : L->sx;
    StraddleJob wp{};
    long long extra = 0;
    if (straddle_in_use(L) && straddle_stale(L, st)) {
        // the GEMM that consumes these slabs reads the straddle block of the same max_4bit_ch
        wp.wst = L->wst; wp.w8m = L->w8m; wp.w8 = L->w8;
        wp.rows = L->N * L->R * L->S;
        wp.C = L->C;
        wp.BK = choose_bk(L);
        wp.blk0 = (L->K_lo / wp.BK) * wp.BK;
        wp.K_lo = L->K_lo;
        extra = ((long long)wp.rows * (wp.BK >> 4) + threads - 1) / threads;
    }
    wp.first_block = (unsigned)extra;   // the straddle blocks come first
    if (dynamic && masked) {
        long long want2 = (M * (L->K_lo / 16) + threads - 1) / threads;
        long long blocks2 = want2 < (long long)sms * 16 ? want2 : (long long)sms * 16;
        if (blocks2 < 1) blocks2 = 1;   // the positions are written even when no group is low
        FLEXIQ_CUDA_TRY(launch_pdl(lower_inplace_kernel, (unsigned)(blocks2 + extra), threads, 0, st, reinterpret_cast<int8_t *>(X4), M, K, G, L->K_lo,
                                   static_cast<const unsigned *>(scratch), sx_out, wp));
        if (wp.wst) straddle_written(L, st);
        record_slab(L, X4, L->K_lo);
        return FLEXIQ_OK;
    }
    const unsigned grid = (unsigned)(blocks + extra);
    if (!masked)
        FLEXIQ_CUDA_TRY(launch_pdl(quantize_lower_kernel<DTYPE, 1>, grid, threads, 0, st, X, M, K, G, L->K_lo, S, L->perm, sx, scratch, X4, pitch, X8, pitch8, dynamic ? sx_out : nullptr, wp));
    else
        FLEXIQ_CUDA_TRY(launch_pdl(quantize_lower_kernel<DTYPE, 0>, grid, threads, 0, st, X, M, K, G, L->K_lo, S, L->perm, sx, scratch, X4, pitch, X8, pitch8, dynamic ? sx_out : nullptr, wp));
    if (extra) straddle_written(L, st);
    // remember at which max_4bit_ch these buffers were written (the mixed_* calls check it)
    if (masked || L->K_lo > 0) record_slab(L, X4, L->K_lo);
    if (!masked && L->K_lo < L->C) record_slab(L, X8, L->K_lo);
    return FLEXIQ_OK;
}

}  // namespace flexiq

using namespace flexiq;

extern "C" int flexiq_quantize_lower(flexiq_layer_t layer, const void *X_dev, int x_dtype, int64_t M, float x_scale,
                                     int dynamic_pos, uint8_t *X4_dev, int8_t *X8_dev, uint8_t *x_shift_out_dev,
                                     uint32_t *scratch_dev, void *stream)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (M < 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "M = %lld is negative", (long long)M);
    if (x_dtype < FLEXIQ_DTYPE_F32 || x_dtype > FLEXIQ_DTYPE_I8)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "unknown x_dtype %d", x_dtype);
    if (x_dtype != FLEXIQ_DTYPE_I8 && !(x_scale > 0.0f))
        return set_error(FLEXIQ_ERR_INVALID_ARG, "x_scale %g must be positive", (double)x_scale);
    if (M == 0) return FLEXIQ_OK;
    const int K_lo = L->K_lo, K_hi = L->C - K_lo;
    if (!X_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "X_dev is NULL");
    const bool packed = L->lowbit_path == FLEXIQ_LOWBIT_PACKED_U4;
    if (!packed && !X4_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "X4_dev is NULL: on the masked path it is the whole slab [M][K]");
    if (packed && K_lo > 0 && !X4_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "X4_dev is NULL but K_lo = %d", K_lo);
    if (packed && K_hi > 0 && !X8_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "X8_dev is NULL but K_hi = %d", K_hi);
    if (dynamic_pos && (!x_shift_out_dev || !scratch_dev))
        return set_error(FLEXIQ_ERR_INVALID_ARG, "dynamic_pos needs x_shift_out_dev and scratch_dev");
    if ((reinterpret_cast<uintptr_t>(X_dev) | reinterpret_cast<uintptr_t>(X4_dev) | reinterpret_cast<uintptr_t>(X8_dev)) & 15)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "X_dev, X4_dev and X8_dev must be 16-byte aligned");
    int rc = check_device_sm100();
    if (rc) return rc;
    if ((rc = check_layer_device(L))) return rc;
    int64_t pitch = 0;
    flexiq_x4_pitch(layer, K_lo, &pitch);
    // masked path: one slab, low groups first, the 8-bit groups behind them in the same rows
    long long pitch8 = K_hi;
    if (!packed) { X8_dev = reinterpret_cast<int8_t *>(X4_dev) + K_lo; pitch8 = L->C; }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    switch (x_dtype) {
        case FLEXIQ_DTYPE_F32: return launch_prologue<FLEXIQ_DTYPE_F32>(L, X_dev, M, x_scale, dynamic_pos, X4_dev, pitch, X8_dev, pitch8, x_shift_out_dev, scratch_dev, st);
        case FLEXIQ_DTYPE_F16: return launch_prologue<FLEXIQ_DTYPE_F16>(L, X_dev, M, x_scale, dynamic_pos, X4_dev, pitch, X8_dev, pitch8, x_shift_out_dev, scratch_dev, st);
        case FLEXIQ_DTYPE_BF16: return launch_prologue<FLEXIQ_DTYPE_BF16>(L, X_dev, M, x_scale, dynamic_pos, X4_dev, pitch, X8_dev, pitch8, x_shift_out_dev, scratch_dev, st);
        default: return launch_prologue<FLEXIQ_DTYPE_I8>(L, X_dev, M, x_scale, dynamic_pos, X4_dev, pitch, X8_dev, pitch8, x_shift_out_dev, scratch_dev, st);
    }
}

extern "C" int flexiq_quantize_lower_dynamic_noalloc(flexiq_layer_t layer, const void *X_dev, int x_dtype, int64_t M,
                                                     float x_scale, uint8_t *X4_dev, int8_t *X8_dev,
                                                     uint8_t *x_shift_out_dev, void *stream)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (L->n_g > kStaticScratchGroups)
        return set_error(FLEXIQ_ERR_INVALID_ARG,
                         "layer has %d channel groups; the built-in scratch of this entry point holds at most %d "
                         "(use flexiq_quantize_lower with caller-provided scratch instead)", L->n_g, kStaticScratchGroups);
    int rc = check_layer_device(L);   // the array's address is per device: look it up on the layer's
    if (rc) return rc;
    unsigned *scratch = nullptr;
    if ((rc = static_scratch_address(&scratch))) return rc;
    return flexiq_quantize_lower(layer, X_dev, x_dtype, M, x_scale, 1, X4_dev, X8_dev, x_shift_out_dev, scratch, stream);
}

// Mixed-precision GEMM / implicit-GEMM convolution mainloop and epilogue (Sec. 7):
//   acc = sum over low groups of (4-bit dot products) << positions + 8-bit dot products,
// exact in int32, then the per-output-channel epilogue.
//
// Design for sm_100a.  The 4-bit values, shifted back to their extraction positions, are
// 8-bit integers (|x4 << sx| <= 128), so low and high channel groups feed ONE chain of
// tcgen05.mma.kind::i8 instructions accumulating in TMEM: no per-group round trip through
// registers for the shift.  A persistent, warp-specialised CTA per SM:
//   warp 0      TMA producer (tiled loads for linear layers, im2col loads for convs)
//   warp 1      TMEM allocation + single-thread MMA issue
//   warps 2..5  epilogue: tcgen05.ld, scale / bias / round / clip, 128-bit stores
//   warps 6..9  (packed low-bit path only) widen 4-bit slabs to 8-bit operands in smem
// Two TMEM accumulators let the epilogue of tile i overlap the mainloop of tile i+1.
// Every wait is bounded; an expired wait raises the status word and the CTA drains.
#include "flexiq_internal.h"
#include "sm100_ptx.cuh"

namespace flexiq {

__device__ unsigned int g_status_word = 0;

constexpr int BM = 128;
constexpr int kNumEpiWarps = 4;
constexpr int kThreadsMasked = 32 * (2 + kNumEpiWarps);
constexpr uint32_t kSpinLimit = 1u << 22;

struct GemmParams {
    long long M;         // rows of the implicit GEMM (tokens or output pixels)
    int N;               // output channels
    int C;               // channels per tap
    int C_lo, C_hi;      // max_4bit_ch and the rest
    int T, S;            // taps R*S and S
    int BK;              // K bytes per stage: 128 or 64
    int nb_lo, nb_hi;    // k-blocks per tap in the low / high slab
    int im2col;          // A operand through im2col-mode TMA
    int P, Q, stride, pad;
    int out_mode;
    float x_scale, y_scale;
    const float *w_scale;
    const float *bias;
    void *Y;
    int m_tiles, n_tiles;
};

template <int BN>
struct Cfg {
    static constexpr int kStages = BN == 256 ? 4 : (BN == 128 ? 6 : 8);
    static constexpr int kABytes = BM * 128;
    static constexpr int kBBytes = BN * 128;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTmemCols = 2 * BN;
    // stages | alpha/beta [2][BN] each | barriers | tmem ptr, abort flag
    static constexpr int kSmemBytes = kStages * kStageBytes + 4 * BN * 4 + (2 * kStages + 4) * 8 + 16 + 1024;
};

// Bounded wait.  Returns false after the limit or when another role already gave up;
// the caller then leaves its loops and the CTA drains.
__device__ __forceinline__ bool wait_bounded(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int where)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (it > 64) {
            if (*abort_flag) return false;
            __nanosleep(it > 4096 ? 256 : 32);
        }
    }
    *abort_flag = 1;
    atomicMax(&g_status_word, 0x100u + (unsigned)where);
    return false;
}

// All epilogue threads agree on whether the wait succeeded, so that no warp runs ahead
// to the next tile's barrier while another one has left the loop.
__device__ __forceinline__ bool epilogue_vote(bool ok)
{
    uint32_t all;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.u32 p, %1, 0;\n"
        "bar.red.and.pred q, 2, %2, p;\n"
        "selp.u32 %0, 1, 0, q;\n"
        "}\n"
        : "=r"(all)
        : "r"((uint32_t)ok), "n"(32 * kNumEpiWarps)
        : "memory");
    return all != 0;
}

__device__ __forceinline__ unsigned pack4_sat_i8(float y0, float y1, float y2, float y3)
{
    const int a = max(-128, min(127, __float2int_rn(y0)));
    const int b = max(-128, min(127, __float2int_rn(y1)));
    const int c = max(-128, min(127, __float2int_rn(y2)));
    const int d = max(-128, min(127, __float2int_rn(y3)));
    return (unsigned)(a & 0xff) | ((unsigned)(b & 0xff) << 8) | ((unsigned)(c & 0xff) << 16) | ((unsigned)d << 24);
}

template <int BN>
__global__ void __launch_bounds__(kThreadsMasked, 1)
mixed_gemm_kernel(const __grid_constant__ CUtensorMap mapA_lo, const __grid_constant__ CUtensorMap mapA_hi,
                  const __grid_constant__ CUtensorMap mapB_lo, const __grid_constant__ CUtensorMap mapB_hi,
                  const GemmParams p)
{
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *stage_base = smem;
    float *alpha_s = reinterpret_cast<float *>(smem + C::kStages * C::kStageBytes);  // [2][BN]
    float *beta_s = alpha_s + 2 * BN;                                               // [2][BN]
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(beta_s + 2 * BN);
    uint64_t *empty_bar = full_bar + C::kStages;
    uint64_t *tmem_full = empty_bar + C::kStages;
    uint64_t *tmem_empty = tmem_full + 2;
    uint32_t *tmem_ptr_s = reinterpret_cast<uint32_t *>(tmem_empty + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_ptr_s + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.m_tiles * p.n_tiles;
    const int kb_lo = p.T * p.nb_lo, kb_total = p.T * (p.nb_lo + p.nb_hi);

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            ptx::mbar_init(&full_bar[s], 1);
            ptx::mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&tmem_full[b], 1);
            ptx::mbar_init(&tmem_empty[b], 32 * kNumEpiWarps);
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_ptr_s, C::kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_s;

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer
        if (lane == 0) {
            ptx::prefetch_tmap(&mapA_lo);
            ptx::prefetch_tmap(&mapA_hi);
            ptx::prefetch_tmap(&mapB_lo);
            ptx::prefetch_tmap(&mapB_hi);
            const uint32_t tx_bytes = (uint32_t)(BM * p.BK + BN * p.BK);
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m_blk = tile / p.n_tiles, n_blk = tile - m_blk * p.n_tiles;
                const long long m0 = (long long)m_blk * BM;
                const int n0 = n_blk * BN;
                int pix_w = 0, pix_h = 0, pix_n = 0;
                if (p.im2col) {
                    const long long pq = (long long)p.P * p.Q;
                    pix_n = (int)(m0 / pq);
                    const int rem = (int)(m0 - (long long)pix_n * pq);
                    pix_h = (rem / p.Q) * p.stride - p.pad;
                    pix_w = (rem % p.Q) * p.stride - p.pad;
                }
                for (int kb = 0; kb < kb_total; ++kb) {
                    if (!wait_bounded(&empty_bar[stage], phase ^ 1, abort_flag, 1)) { ok = false; break; }
                    const bool low = kb < kb_lo;
                    const int kk = low ? kb : kb - kb_lo;
                    const int nb = low ? p.nb_lo : p.nb_hi;
                    const int tap = kk / nb, cb = kk - tap * nb;
                    uint8_t *sa = stage_base + stage * C::kStageBytes;
                    uint8_t *sb = sa + C::kABytes;
                    ptx::mbar_expect_tx(&full_bar[stage], tx_bytes);
                    const CUtensorMap *ma = low ? &mapA_lo : &mapA_hi;
                    if (p.im2col)
                        ptx::tma_load_im2col_4d(sa, ma, &full_bar[stage], cb * p.BK, pix_w, pix_h, pix_n,
                                                (uint16_t)(tap % p.S), (uint16_t)(tap / p.S));
                    else
                        ptx::tma_load_2d(sa, ma, &full_bar[stage], cb * p.BK, (int)m0);
                    // weights: slab-order [N][T*C]; the low slab's forms start each tap at channel 0,
                    // the 8-bit form of the high groups at channel C_lo
                    ptx::tma_load_2d(sb, low ? &mapB_lo : &mapB_hi, &full_bar[stage],
                                     tap * p.C + (low ? 0 : p.C_lo) + cb * p.BK, n0);
                    ++issued;
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                // drain: let the copies already in flight land before the CTA retires
                const int n_back = issued < C::kStages ? (int)issued : C::kStages;
                int s = stage;
                uint32_t ph = phase;
                for (int i = 0; i < n_back; ++i) {
                    if (--s < 0) { s = C::kStages - 1; ph ^= 1; }
                    for (uint32_t it = 0; it < (1u << 16); ++it) {
                        if (ptx::mbar_try_wait(&full_bar[s], ph)) break;
                        __nanosleep(64);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = ptx::idesc_i8(BM, BN);
            int stage = 0;
            uint32_t phase = 0;
            int buf = 0;
            uint32_t buf_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                if (!wait_bounded(&tmem_empty[buf], buf_phase ^ 1, abort_flag, 2)) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < kb_total; ++kb) {
                    if (!wait_bounded(&full_bar[stage], phase, abort_flag, 3)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const bool low = kb < kb_lo;
                    const int kk = low ? kb : kb - kb_lo;
                    const int nb = low ? p.nb_lo : p.nb_hi;
                    const int cb = kk % nb;
                    const int valid = min(p.BK, (low ? p.C_lo : p.C_hi) - cb * p.BK);
                    const int ksteps = (valid + 31) >> 5;
                    const uint32_t sa = ptx::smem_u32(stage_base + stage * C::kStageBytes);
                    const uint64_t adesc = ptx::smem_desc(sa, p.BK);
                    const uint64_t bdesc = ptx::smem_desc(sa + C::kABytes, p.BK);
                    for (int k = 0; k < ksteps; ++k)  // 32 bytes of K per instruction: +2 in 16-byte units
                        ptx::mma_i8(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
                    ptx::mma_commit(&empty_bar[stage]);
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                }
                if (ok) ptx::mma_commit(&tmem_full[buf]);
                if ((buf ^= 1) == 0) buf_phase ^= 1;
            }
        }
    } else {
        // ------------------------------------------------------------- epilogue
        const int quad = warp & 3;  // TMEM lane quadrant this warp may read
        const int et = threadIdx.x - 64;
        int buf = 0;
        uint32_t buf_phase = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
            const int m_blk = tile / p.n_tiles, n_blk = tile - m_blk * p.n_tiles;
            const int n0 = n_blk * BN;
            // per-output-channel factors of this tile: alpha = (S_x * S_w) / S_y, beta = bias / S_y
            for (int c = et; c < BN; c += 32 * kNumEpiWarps) {
                const int n = n0 + c;
                float a = 0.f, b = 0.f;
                if (n < p.N) {
                    const float sxw = __fmul_rn(p.x_scale, p.w_scale[n]);
                    const float bv = p.bias ? p.bias[n] : 0.f;
                    if (p.out_mode == FLEXIQ_OUT_REQUANT_I8) {
                        a = __fdiv_rn(sxw, p.y_scale);
                        b = __fdiv_rn(bv, p.y_scale);
                    } else {
                        a = sxw;
                        b = bv;
                    }
                }
                alpha_s[buf * BN + c] = a;
                beta_s[buf * BN + c] = b;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kNumEpiWarps) : "memory");
            if (!epilogue_vote(wait_bounded(&tmem_full[buf], buf_phase, abort_flag, 4))) break;
            ptx::tc_fence_after_sync();
            const long long m = (long long)m_blk * BM + quad * 32 + lane;
            const bool row_ok = m < p.M;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BN);
            const float *al = alpha_s + buf * BN, *be = beta_s + buf * BN;
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                ptx::tmem_ld_32x32(taddr + c, r);
                ptx::tmem_ld_wait();
                const int n = n0 + c;
                if (row_ok && n < p.N) {
                    const bool second = n + 16 < p.N;  // N is a multiple of 16
                    if (p.out_mode == FLEXIQ_OUT_REQUANT_I8) {
                        unsigned w[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            w[i] = pack4_sat_i8(fmaf((float)(int)r[4 * i + 0], al[c + 4 * i + 0], be[c + 4 * i + 0]),
                                                fmaf((float)(int)r[4 * i + 1], al[c + 4 * i + 1], be[c + 4 * i + 1]),
                                                fmaf((float)(int)r[4 * i + 2], al[c + 4 * i + 2], be[c + 4 * i + 2]),
                                                fmaf((float)(int)r[4 * i + 3], al[c + 4 * i + 3], be[c + 4 * i + 3]));
                        uint4 *dst = reinterpret_cast<uint4 *>(static_cast<int8_t *>(p.Y) + m * p.N + n);
                        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                        if (second) dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                    } else if (p.out_mode == FLEXIQ_OUT_DEQUANT_F32) {
                        float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(p.Y) + m * p.N + n);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            if (i >= 4 && !second) break;
                            dst[i] = make_float4(fmaf((float)(int)r[4 * i + 0], al[c + 4 * i + 0], be[c + 4 * i + 0]),
                                                 fmaf((float)(int)r[4 * i + 1], al[c + 4 * i + 1], be[c + 4 * i + 1]),
                                                 fmaf((float)(int)r[4 * i + 2], al[c + 4 * i + 2], be[c + 4 * i + 2]),
                                                 fmaf((float)(int)r[4 * i + 3], al[c + 4 * i + 3], be[c + 4 * i + 3]));
                        }
                    } else {
                        uint4 *dst = reinterpret_cast<uint4 *>(static_cast<int32_t *>(p.Y) + m * p.N + n);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            if (i >= 4 && !second) break;
                            dst[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
                        }
                    }
                }
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&tmem_empty[buf]);
            if ((buf ^= 1) == 0) buf_phase ^= 1;
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

// ------------------------------------------------------------------------------------
// host side

static int bn_index(int bn) { return bn == 64 ? 0 : (bn == 128 ? 1 : 2); }

// Tile width: fewest machine-waves weighted by how well a tile of that width feeds the
// tensor pipe (narrow tiles re-read A from shared memory more often per MMA).
int choose_bn(long long m_tiles, int N, int sms)
{
    const int bns[3] = {256, 128, 64};
    const double penalty[3] = {1.0, 1.15, 1.6};
    int best = 256;
    double best_cost = 1e300;
    for (int i = 0; i < 3; ++i) {
        const long long n_tiles = (N + bns[i] - 1) / bns[i];
        const long long tiles = m_tiles * n_tiles;
        const long long waves = (tiles + sms - 1) / sms;
        const double cost = (double)waves * bns[i] * penalty[i];
        if (cost < best_cost - 1e-9) { best_cost = cost; best = bns[i]; }
    }
    return best;
}

static int make_map_im2col(CUtensorMap *map, const void *base, int Cpart, long long pitch, int Nb, int H, int W,
                           int R, int S, int stride, int pad, int bk)
{
    EncodeIm2colFn enc = get_encode_im2col();
    if (!enc) return set_error(FLEXIQ_ERR_CUDA, "cuTensorMapEncodeIm2col is not available from the driver");
    if ((reinterpret_cast<uintptr_t>(base) & 15) != 0 || (pitch & 15) != 0)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "conv slab base %p / pixel pitch %lld not 16-byte aligned", base, pitch);
    cuuint64_t dims[4] = {(cuuint64_t)Cpart, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)Nb};
    cuuint64_t strides[3] = {(cuuint64_t)pitch, (cuuint64_t)pitch * W, (cuuint64_t)pitch * W * H};
    int lower[2] = {-pad, -pad};
    int upper[2] = {pad - (S - 1), pad - (R - 1)};
    cuuint32_t estr[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), dims, strides, lower, upper,
                     (cuuint32_t)bk, (cuuint32_t)BM, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     bk == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return set_error(FLEXIQ_ERR_CUDA, "cuTensorMapEncodeIm2col failed with CUresult %d", (int)r);
    return FLEXIQ_OK;
}

template <int BN>
static int launch_bn(const CUtensorMap &a_lo, const CUtensorMap &a_hi, const CUtensorMap &b_lo, const CUtensorMap &b_hi,
                     const GemmParams &p, int sms, cudaStream_t st)
{
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 64 && !attr_set[dev]) {
        FLEXIQ_CUDA_TRY(cudaFuncSetAttribute(mixed_gemm_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BN>::kSmemBytes));
        attr_set[dev] = true;
    }
    const long long tiles = (long long)p.m_tiles * p.n_tiles;
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    mixed_gemm_kernel<BN><<<grid, kThreadsMasked, Cfg<BN>::kSmemBytes, st>>>(a_lo, a_hi, b_lo, b_hi, p);
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    return FLEXIQ_OK;
}

static int run_mixed(Layer *L, const uint8_t *X4, const int8_t *X8, const uint8_t *x_shift, long long M, int Nb, int H,
                     int W, float x_scale, float y_scale, int out_mode, void *Y, cudaStream_t st)
{
    (void)x_shift;
    if (out_mode < FLEXIQ_OUT_ACC_I32 || out_mode > FLEXIQ_OUT_DEQUANT_F32)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "unknown out_mode %d", out_mode);
    if (out_mode == FLEXIQ_OUT_REQUANT_I8 && !(y_scale > 0.0f))
        return set_error(FLEXIQ_ERR_INVALID_ARG, "y_scale %g must be positive", (double)y_scale);
    if (M == 0) return FLEXIQ_OK;
    const int C_lo = L->K_lo, C_hi = L->C - C_lo;
    if (!Y) return set_error(FLEXIQ_ERR_INVALID_ARG, "Y_dev is NULL");
    if (C_lo > 0 && !X4) return set_error(FLEXIQ_ERR_INVALID_ARG, "X4_dev is NULL but K_lo = %d", C_lo);
    if (C_hi > 0 && !X8) return set_error(FLEXIQ_ERR_INVALID_ARG, "X8_dev is NULL but K_hi = %d", C_hi);
    if ((reinterpret_cast<uintptr_t>(Y) | reinterpret_cast<uintptr_t>(X4) | reinterpret_cast<uintptr_t>(X8)) & 15)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "X4_dev, X8_dev and Y_dev must be 16-byte aligned");
    if (L->lowbit_path != FLEXIQ_LOWBIT_MASKED_I8)
        return set_error(FLEXIQ_ERR_UNSUPPORTED, "packed low-bit mainloop is not available in this build");
    int rc = check_device_sm100();
    if (rc) return rc;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, L->device);

    GemmParams p{};
    p.M = M; p.N = L->N; p.C = L->C; p.C_lo = C_lo; p.C_hi = C_hi;
    p.T = L->R * L->S; p.S = L->S;
    p.BK = choose_bk(L);
    p.nb_lo = (C_lo + p.BK - 1) / p.BK;
    p.nb_hi = (C_hi + p.BK - 1) / p.BK;
    p.im2col = L->is_conv && (L->R != 1 || L->S != 1 || L->stride != 1 || L->pad != 0);
    p.stride = L->stride; p.pad = L->pad;
    if (L->is_conv) {
        p.P = (H + 2 * L->pad - L->R) / L->stride + 1;
        p.Q = (W + 2 * L->pad - L->S) / L->stride + 1;
    }
    p.out_mode = out_mode; p.x_scale = x_scale; p.y_scale = y_scale;
    p.w_scale = L->w_scale; p.bias = L->bias; p.Y = Y;
    p.m_tiles = (int)((M + BM - 1) / BM);
    const int bn = choose_bn(p.m_tiles, L->N, sms);
    p.n_tiles = (L->N + bn - 1) / bn;

    // activation maps (per call: they depend on the caller's buffers, M and the ratio);
    // an empty slab borrows the other one's map and is never addressed
    CUtensorMap a_lo, a_hi;
    const long long pitch_lo = C_lo;  // masked path: one int8 per value
    if (p.im2col) {
        if (C_lo > 0 && (rc = make_map_im2col(&a_lo, X4, C_lo, pitch_lo, Nb, H, W, L->R, L->S, L->stride, L->pad, p.BK))) return rc;
        if (C_hi > 0 && (rc = make_map_im2col(&a_hi, X8, C_hi, C_hi, Nb, H, W, L->R, L->S, L->stride, L->pad, p.BK))) return rc;
    } else {
        const long long rows = L->is_conv ? (long long)Nb * H * W : M;
        if (C_lo > 0 && (rc = make_map_2d(&a_lo, X4, (uint64_t)C_lo, (uint64_t)rows, (uint64_t)pitch_lo, p.BK, BM, p.BK))) return rc;
        if (C_hi > 0 && (rc = make_map_2d(&a_hi, X8, (uint64_t)C_hi, (uint64_t)rows, (uint64_t)C_hi, p.BK, BM, p.BK))) return rc;
    }
    if (C_lo == 0) a_lo = a_hi;
    if (C_hi == 0) a_hi = a_lo;
    const int bi = bn_index(bn);
    switch (bn) {
        case 256: return launch_bn<256>(a_lo, a_hi, L->map_w8m[bi], L->map_w8[bi], p, sms, st);
        case 128: return launch_bn<128>(a_lo, a_hi, L->map_w8m[bi], L->map_w8[bi], p, sms, st);
        default: return launch_bn<64>(a_lo, a_hi, L->map_w8m[bi], L->map_w8[bi], p, sms, st);
    }
}

}  // namespace flexiq

using namespace flexiq;

extern "C" int flexiq_mixed_gemm(flexiq_layer_t layer, const uint8_t *X4_dev, const int8_t *X8_dev,
                                 const uint8_t *x_shift_dev, int64_t M, float x_scale, float y_scale, int out_mode,
                                 void *Y_dev, void *stream)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (L->is_conv) return set_error(FLEXIQ_ERR_INVALID_ARG, "layer is a convolution: use flexiq_mixed_conv");
    if (M < 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "M = %lld is negative", (long long)M);
    return run_mixed(L, X4_dev, X8_dev, x_shift_dev, M, 0, 0, 0, x_scale, y_scale, out_mode, Y_dev,
                     reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int flexiq_mixed_conv(flexiq_layer_t layer, const uint8_t *X4_dev, const int8_t *X8_dev,
                                 const uint8_t *x_shift_dev, int Nb, int H, int W, float x_scale, float y_scale,
                                 int out_mode, void *Y_dev, void *stream)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (!L->is_conv) return set_error(FLEXIQ_ERR_INVALID_ARG, "layer is linear: use flexiq_mixed_gemm");
    if (Nb < 0 || H <= 0 || W <= 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "bad activation shape Nb=%d H=%d W=%d", Nb, H, W);
    const int P = (H + 2 * L->pad - L->R) / L->stride + 1;
    const int Q = (W + 2 * L->pad - L->S) / L->stride + 1;
    if (P <= 0 || Q <= 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "filter does not fit the padded input");
    return run_mixed(L, X4_dev, X8_dev, x_shift_dev, (long long)Nb * P * Q, Nb, H, W, x_scale, y_scale, out_mode, Y_dev,
                     reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int flexiq_check_status(void *stream)
{
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    unsigned int word = 0, zero = 0;
    FLEXIQ_CUDA_TRY(cudaStreamSynchronize(st));
    FLEXIQ_CUDA_TRY(cudaMemcpyFromSymbol(&word, g_status_word, sizeof(word)));
    if (word != 0) {
        FLEXIQ_CUDA_TRY(cudaMemcpyToSymbol(g_status_word, &zero, sizeof(zero)));
        return set_error(FLEXIQ_ERR_TIMEOUT, "a bounded device-side wait expired (status word 0x%x)", word);
    }
    return FLEXIQ_OK;
}

// Mixed-precision GEMM / implicit-GEMM convolution mainloop and epilogue (Sec. 7):
//   acc = sum over low groups of (4-bit dot products) << positions + 8-bit dot products,
// exact in int32, then the per-output-channel epilogue.
//
// Design for sm_100a.  The 4-bit values, shifted back to their extraction positions, are
// 8-bit integers (|x4 << sx| <= 128), so low and high channel groups feed ONE chain of
// tcgen05.mma.kind::i8 instructions accumulating in TMEM: no per-group round trip through
// registers for the shift.  A persistent, warp-specialised CTA per SM, or a CTA pair (cluster of two,
// cta_group::2) per 256-row tile:
//   warp 0       TMA producer (tiled loads for linear layers, im2col loads for convs)
//   warp 1, 18   MMA issue (one elected lane each), tiles taken in turn with one accumulator each; warp 1
//                also allocates TMEM (on the packed path warp 1 issues alone)
//   warps 2..17  epilogue, four per TMEM lane quadrant: tcgen05.ld, scale / bias / round / clip, the
//                results staged in shared memory 32 rows x 32 bytes at a time and written by tiled bulk
//                stores (the fused boundary in original channel order scatters 16-byte chunks directly);
//                on the packed path eight of them widen 4-bit tiles instead
// Two TMEM accumulators let the epilogue of tile i overlap the mainloop of tile i+1.  Launches of one narrow,
// long-K tile per CTA instead let the two MMA warps share the tile's K blocks (an accumulator each, summed
// in the epilogue).
// Every wait is bounded; an expired wait raises the status word and the CTA drains.
#include "flexiq_internal.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "sm100_ptx.cuh"
#include "straddle.cuh"
#include "role_timers.cuh"   // PROF_* expand to nothing in the product build

namespace flexiq {

__device__ unsigned int g_status_word = 0;


constexpr int BM = 128;
constexpr int kNumWorkWarps = 16;                     // epilogue warps (+ expander warps on the packed path)
constexpr int kThreads = 32 * (3 + kNumWorkWarps);      // producer, two MMA warps (the second one last), work warps
constexpr int kRawStages = 2;                         // packed path: ring of raw 4-bit tiles in front of the operand ring
constexpr uint32_t kSpinLimit = 1u << 21;              // parked waits of <= 1 us each: about two seconds at most
constexpr int kStageRegion = 196608;                  // shared memory given to the operand ring
constexpr int kFactorsPerWarp = 512;                  // alpha[64] | beta[64] of the warp's columns in the current tile
constexpr int kMaxStages = 8;
constexpr int kStoreStagePerWarp = 1024;              // 32 rows x 32 int8 columns staged for a tiled bulk store
constexpr int kSmemBytes = kStageRegion + kNumWorkWarps * (kFactorsPerWarp + kStoreStagePerWarp) + 256;

// Internal epilogue mode of the fused layer boundary: the int8 result goes straight into the
// next layer's masked slab (its channel order, its low groups lowered).
constexpr int kOutNextSlab = 3;

struct GemmParams {
    long long M;         // rows of the implicit GEMM (tokens or output pixels)
    int N;               // output channels
    int C;               // channels per tap
    int C_lo, C_hi;      // max_4bit_ch and the rest
    int T, S;            // taps R*S and S
    int BK;              // K bytes per stage: 128 or 64
    int BN;              // tile width: 64, 128, 192 or 256
    int stages;          // depth of the operand ring
    int tps;             // filter taps per ring stage (> 1 only for masked convolutions whose C fits one K block)
    int nb_lo, nb_hi;    // K blocks per tap of the first / second run of blocks (packed path: low slab / 8-bit slab;
                         // masked path: blocks read from w8m plus the straddle block / blocks read from w8)
    int ks_last_lo, ks_last_hi;  // 32-byte K steps of the last block of each run (the others have BK / 32)
    int xa_hi0, xb_hi0;  // first A / B column of the second run within a tap
    int st_cb;           // masked path: block of the first run that is read from the straddle buffer (its last), or -1
    int b_tap_step;      // multi-tap stages: columns from one tap to the next in the weight operand
    int im2col;          // A operand through im2col-mode TMA
    int P, Q, stride, pad;
    int out_mode;
    const float *alpha;  // [N] per-output-channel multiplier of this call
    const float *beta;   // [N] per-output-channel addend of this call
    void *Y;
    int m_tiles, n_tiles;
    // fused layer boundary only: where each 16-channel chunk of the output lands in the next layer's slab
    const int32_t *next_ent;   // [N/16] slab position (in chunks) of original chunk c | its group's position << 24
    int next_K_lo;             // the next layer's max_4bit_ch
    int relu;                  // clamp at zero before the re-quantization
    int tma_store;             // int8 output leaves through shared memory and tiled bulk stores (mapY)
    // Resident weights (convolutions on the multi-tap path whose output channels fit one tile): every tap's
    // weight tile is loaded once per CTA and stays in shared memory in front of the ring, whose stages then hold
    // activation taps only: half as many copies per tile for the producer lane, which bounds these layers.
    int b_res;
    // Patch mode (KIND 2: 3x3-like convolutions of stride 1 whose channels fit one K block and whose output
    // channels fit one tile): a tile is TH = 128 / PW whole output rows of one image, its 128 accumulator rows
    // being the positions y * PW + x of a grid whose pitch PW (a power of two >= W + pad) leaves a few unused
    // columns.  The input patch of TH + R - 1 rows x PW pixels is loaded ONCE per tile by a tiled 4-D copy
    // (halo and padding arrive as zeros); filter tap (r, s) is the same patch read from row offset r * PW + s,
    // so every input pixel crosses from L2 once instead of R * S times.  When W + 2 pad > PW the rightmost taps of the
    // last pixels of an output row index a column beyond the pitch, i.e. the first columns of the NEXT patch row: that
    // is its left padding, zeros, which is what the right padding should read -- provided the row exists, so the
    // patch then carries one more row.
    int pw_log2, TH, tiles_per_img, patch_stage;   // patch_stage: bytes of one ring stage (the patch, rounded up to 1 KB)
    int patch_rows;      // input rows of a patch: TH + R - 1, plus one when a tap's column index can pass the pitch (see above)
    // packed low-bit path only: positions the expander warps shift the 4-bit values back to
    const uint8_t *sx;   // [n_g] activation positions, slab order
    const uint8_t *sw;   // [n_g][N] weight positions
    int G;               // channel-group size
};

// Bounded wait.  Returns false after the limit or when another role already gave up;
// the caller then leaves its loops and the CTA drains.  The slow path stays out of line
// so that the hot loops remain small.
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag, int where, uint32_t limit = kSpinLimit)
{
    // a few quick polls for the common short wait, then hardware-parked waits of up to a
    // microsecond each: they wake at once when the phase completes and issue nothing meanwhile
    for (uint32_t it = 0; it < 8; ++it)
        if (ptx::mbar_try_wait_s(bar, parity)) return true;
    for (uint32_t it = 0; it < limit; ++it) {
        if (ptx::mbar_try_wait_hint_s(bar, parity, 1000u)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    atomicMax(&g_status_word, 0x100u + (unsigned)where);
    return false;
}
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int *abort_flag, int where)
{
    if (ptx::mbar_try_wait_s(bar, parity)) return true;
    return wait_slow(bar, parity, abort_flag, where);
}
__device__ __forceinline__ bool wait_bounded(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int where)
{
    return wait_bounded(ptx::smem_u32(bar), parity, abort_flag, where);
}

// Static round-robin walk over the output tiles of one CTA (or CTA pair) without divisions
// in the loop: tile = first + i * step, decoded as (m_blk, n_blk).
struct TileWalk {
    int m_blk, n_blk, step_m, step_n, n_tiles, left;
    __device__ __forceinline__ void init(int first, int step, int num_tiles, int n_tiles_)
    {
        n_tiles = n_tiles_;
        m_blk = first / n_tiles;
        n_blk = first - m_blk * n_tiles;
        step_m = step / n_tiles;
        step_n = step - step_m * n_tiles;
        left = first < num_tiles ? (num_tiles - first + step - 1) / step : 0;
    }
    __device__ __forceinline__ void next()
    {
        --left;
        m_blk += step_m;
        n_blk += step_n;
        if (n_blk >= n_tiles) { n_blk -= n_tiles; ++m_blk; }
    }
};

// Output pixel coordinates (image n, row h, column w) of a running row index that advances by a fixed
// number of rows per step, plus one block of rows when the tile walk wraps to the next block row.
struct PixelWalk {
    int n, h, w;
    int dn, dh, dw, en, eh, ew;
    __device__ __forceinline__ static void split(long long idx, int P, int Q, int &n_, int &h_, int &w_)
    {
        const long long pq = (long long)P * Q;
        n_ = (int)(idx / pq);
        const int rem = (int)(idx - (long long)n_ * pq);
        h_ = rem / Q;
        w_ = rem - h_ * Q;
    }
    __device__ __forceinline__ void init(long long first_row, long long step_rows, long long block_rows, int P, int Q)
    {
        split(first_row, P, Q, n, h, w);
        split(step_rows, P, Q, dn, dh, dw);
        split(block_rows, P, Q, en, eh, ew);
    }
    __device__ __forceinline__ void add(int an, int ah, int aw, int P, int Q)
    {
        w += aw;
        if (w >= Q) { w -= Q; ++h; }
        h += ah;
        if (h >= P) { h -= P; ++n; }
        n += an;
    }
    // one step of the tile walk that moved to another block row; extra = 1 when it also wrapped
    __device__ __forceinline__ void advance(int extra, int P, int Q)
    {
        add(dn, dh, dw, P, Q);
        if (extra > 0) add(en, eh, ew, P, Q);
    }
};

// two int32 -> two saturated int8 in the low half, upper half taken from c's low half
__device__ __forceinline__ unsigned pack2_sat_s8(int hi, int lo, unsigned c)
{
    unsigned d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(hi), "r"(lo), "r"(c));
    return d;
}
// round-half-even, saturate to int8, pack little-endian (y0 in the lowest byte)
__device__ __forceinline__ unsigned requant4(float y0, float y1, float y2, float y3)
{
    const unsigned top = pack2_sat_s8(__float2int_rn(y3), __float2int_rn(y2), 0u);
    return pack2_sat_s8(__float2int_rn(y1), __float2int_rn(y0), top);
}

// two fp32 -> two fp16 (or bf16) values, round to nearest even, the first in the low half
template <bool BF16> __device__ __forceinline__ uint32_t pack2_f16(float lo, float hi)
{
    if (BF16) {
        const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<const uint32_t *>(&v);
    }
    const __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}

// 16 accumulator columns of one row -> 16 output values, through the per-channel factors.
//   REQUANT_I8 : 16 bytes (one 128-bit word);  DEQUANT_F32 / ACC_I32 : 64 bytes.
template <int MODE>
__device__ __forceinline__ void finish16(const uint32_t *r, const float *alpha16, const float *beta16, uint32_t *out)
{
    const float4 *fa = reinterpret_cast<const float4 *>(alpha16), *fb = reinterpret_cast<const float4 *>(beta16);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (MODE == FLEXIQ_OUT_ACC_I32) {
            out[4 * i + 0] = r[4 * i + 0]; out[4 * i + 1] = r[4 * i + 1]; out[4 * i + 2] = r[4 * i + 2]; out[4 * i + 3] = r[4 * i + 3];
        } else {
            const float4 a = fa[i], b = fb[i];
            const float y0 = fmaf((float)(int)r[4 * i + 0], a.x, b.x), y1 = fmaf((float)(int)r[4 * i + 1], a.y, b.y);
            const float y2 = fmaf((float)(int)r[4 * i + 2], a.z, b.z), y3 = fmaf((float)(int)r[4 * i + 3], a.w, b.w);
            if (MODE == FLEXIQ_OUT_REQUANT_I8) {
                out[i] = requant4(y0, y1, y2, y3);
            } else {
                out[4 * i + 0] = __float_as_uint(y0); out[4 * i + 1] = __float_as_uint(y1);
                out[4 * i + 2] = __float_as_uint(y2); out[4 * i + 3] = __float_as_uint(y3);
            }
        }
    }
}
// Fused layer boundary: 16 outputs re-quantized with the next layer's activation scale, clipped
// to [lo, hi] before the rounding (the range the next layer's 4-bit value can hold at its
// position, or the int8 range), low bits cleared by `mask`: the next layer's masked slab bytes.
__device__ __forceinline__ void finish16_next(const uint32_t *r, const float *alpha16, const float *beta16, float lo, float hi,
                                              uint32_t mask, uint32_t *out)
{
    const float4 *fa = reinterpret_cast<const float4 *>(alpha16), *fb = reinterpret_cast<const float4 *>(beta16);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float4 a = fa[i], b = fb[i];
        const float y0 = fminf(fmaxf(fmaf((float)(int)r[4 * i + 0], a.x, b.x), lo), hi);
        const float y1 = fminf(fmaxf(fmaf((float)(int)r[4 * i + 1], a.y, b.y), lo), hi);
        const float y2 = fminf(fmaxf(fmaf((float)(int)r[4 * i + 2], a.z, b.z), lo), hi);
        const float y3 = fminf(fmaxf(fmaf((float)(int)r[4 * i + 3], a.w, b.w), lo), hi);
        out[i] = requant4(y0, y1, y2, y3) & mask;
    }
}
// One 16-channel chunk of the fused layer boundary.  `ent` = slab position (in chunks) | extraction position << 24.
__device__ __forceinline__ void next_slab16(const GemmParams &p, int ent, const uint32_t *r, const float *alpha16, const float *beta16,
                                            uint32_t *out)
{
    float lo = -128.f, hi = 127.f;
    uint32_t mask = 0xffffffffu;
    if ((ent & 0xffffff) * 16 < p.next_K_lo) {
        const int sft = ent >> 24;
        hi = (float)(8 << sft) - 1.f;
        lo = -(float)(8 << sft);
        mask = ((0xffu << sft) & 0xffu) * 0x01010101u;
    }
    if (p.relu) lo = fmaxf(lo, 0.f);
    // the pack saturates to [-128, 127] by itself: clamp only when the range is narrower (warp-uniform)
    if (lo > -128.f || hi < 127.f) finish16_next(r, alpha16, beta16, lo, hi, mask, out);
    else {
        finish16<FLEXIQ_OUT_REQUANT_I8>(r, alpha16, beta16, out);
#pragma unroll
        for (int q = 0; q < 4; ++q) out[q] &= mask;
    }
}
__device__ __forceinline__ void st_global_128(void *p, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_global_256(void *p, const uint32_t *w)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
}

// Eight packed bytes (16 two's-complement nibbles, channel 2t in bits 0-3 of byte t) -> 16 int8
// values (nibble << s), as four little-endian words.  A nibble n moved to the high half of a byte is the
// int8 value 16 n, and n << s is that byte shifted right arithmetically by 4 - s: a logical shift of the
// whole word (the low halves are zero, so nothing crosses a byte) plus the sign, replicated over each byte
// by a byte permute, in the vacated top bits.
__device__ __forceinline__ void unpack16(uint32_t w0, uint32_t w1, int s, uint32_t out[4])
{
    const uint32_t r = 4u - (uint32_t)s;
    const uint32_t top = 0x01010101u * ((0xff00u >> r) & 0xffu);   // the top r bits of every byte
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t w = h == 0 ? w0 : w1;
        const uint32_t e = (w << 4) & 0xf0f0f0f0u, o = w & 0xf0f0f0f0u;  // even / odd nibbles, each in the high half of a byte
        const uint32_t x[2] = {__byte_perm(e, o, 0x5140), __byte_perm(e, o, 0x7362)};  // channel order
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            uint32_t sign;
            asm("prmt.b32 %0, %1, 0, 0xba98;" : "=r"(sign) : "r"(x[q]));   // 0xff where the byte is negative
            out[2 * h + q] = (x[q] >> r) | (sign & top);
        }
    }
}

// The 9 taps of a 3x3 filter on a halo patch, fully unrolled: tap (r, t) reads the patch from row offset
// r * PW + t (ROW16 sixteen-byte units per pixel row, `down` units per patch row), KS K steps of 32 bytes each.
template <int CG, int ROW16, int KS>
__device__ __forceinline__ void patch_taps_3x3(uint32_t d_tmem, uint32_t a_lo, uint32_t down, uint32_t b_lo, uint32_t b_step,
                                               uint32_t desc_hi, uint32_t idesc)
{
#pragma unroll
    for (int r = 0; r < 3; ++r) {
#pragma unroll
        for (int t = 0; t < 3; ++t) {
#pragma unroll
            for (int k = 0; k < KS; ++k)
                ptx::mma_i8_s<CG>(d_tmem, a_lo + (uint32_t)(t * ROW16 + 2 * k), b_lo + (uint32_t)(2 * k), desc_hi, idesc, (r | t | k) ? 1u : 0u);
            b_lo += b_step;
        }
        a_lo += down;
    }
}

struct EpilogueCtx {
    uint32_t tmem_base, buf_stride, cta_rank;
    uint64_t *tmem_full, *tmem_empty;
    volatile int *abort_flag;
    float *fac;
    uint32_t store_stage;         // this warp's 1 KB of shared memory for staged stores
    const CUtensorMap *map_y, *map_y16;   // boxes of 32 rows x 32 columns (32-byte swizzle) and 32 x 16 (plain)
    int first_tile, tile_step, num_tiles;
    int parts, arrivals_on;  // column parts per tile (4 or 2); this warp arrives on the accumulator barrier
};

// One epilogue warp: TMEM lane quadrant `quad` (32 rows, lane = row), column slot `part` (32 or 64
// columns per pass; two passes when only eight warps drain the tile) of every tile of this CTA.
// Per pass: fetch the columns' factors, read the whole slice of the accumulator into registers,
// hand the accumulator back, then scale / round / clip; the results are staged in shared memory (32 rows
// x 32 bytes: 32 int8, 16 half-precision or 8 four-byte columns) and leave through tiled bulk stores.
template <int CG, int MODE, bool SPLIT, int KIND>
__device__ __forceinline__ void epilogue_role(const GemmParams &p, const EpilogueCtx &x, int quad, int part, int lane)
{
    constexpr bool kPatch = KIND == 2;
    constexpr bool kScaled = MODE != FLEXIQ_OUT_ACC_I32;
    constexpr bool kHalf = MODE == FLEXIQ_OUT_DEQUANT_F16 || MODE == FLEXIQ_OUT_DEQUANT_BF16;
    constexpr int kElem = (MODE == FLEXIQ_OUT_REQUANT_I8 || MODE == kOutNextSlab) ? 1 : (kHalf ? 2 : 4);  // output bytes per element
    const int BN = p.BN;
    // Columns per warp and pass: 64 (tiles of 192 or 256 columns) or 32 (128 or 64), so that every staged
    // box is 32 columns = whole sectors; with 192 or 64 columns the last column slot of a lane quadrant has no
    // columns and its warp only keeps step with the accumulator barriers.
    const int cols = BN >= 192 ? 64 : 32;
    const bool y32 = (reinterpret_cast<uintptr_t>(p.Y) & 31) == 0;
    const bool wide = y32 && (p.N & 31) == 0;    // int8 rows are 32-byte aligned: 256-bit stores
    // lane l keeps factors 4l..4l+3 of the table alpha[64] | beta[64]
    const float *fsrc = (lane < 16 ? p.alpha : p.beta) + 4 * (lane & 15);
    int buf = 0;
    uint32_t buf_phase = 0;
    PROF_DECL(prof_wait);
    PROF_DECL(prof_ld);
    PROF_DECL(prof_math);
    PROF_T0(prof_start);
    const int passes = 4 / x.parts;              // 1 with sixteen epilogue warps, 2 with eight
    // Patch mode keeps four accumulators, tile ti in accumulator ti mod 4.  With 64-column tiles only column
    // slots 0 and 1 of a lane quadrant have columns, so slots 2 and 3 take the odd tiles instead of idling.
    int ti = 0, tile_inc = 1;
    if (kPatch && BN == 64) { tile_inc = 2; ti = part >> 1; part &= 1; }
    TileWalk tw;
    for (tw.init(x.first_tile + ti * x.tile_step, x.tile_step * tile_inc, x.num_tiles, p.n_tiles); tw.left > 0; tw.next(), ti += tile_inc) {
        if (kPatch) { buf = ti & 3; buf_phase = (uint32_t)(ti >> 2) & 1u; }
        long long row = ((long long)tw.m_blk * CG + x.cta_rank) * BM + quad * 32 + lane;
        // where the warp's 32 accumulator rows go: rows row0.. of Y, or in patch mode a box of bx x by pixels
        int st_x = 0, st_y = 0, st_n = 0;
        bool box_live = true;
        if (kPatch) {
            const int pw = 1 << p.pw_log2;
            st_n = tw.m_blk / p.tiles_per_img;
            const int y0 = (tw.m_blk - st_n * p.tiles_per_img) * p.TH;
            const int k = quad * 32 + lane;
            const int yy = y0 + (k >> p.pw_log2), xx = k & (pw - 1);
            row = (yy < p.P && xx < p.Q) ? ((long long)st_n * p.P + yy) * p.Q + xx : p.M;   // p.M: not an output pixel
            st_y = y0 + ((quad * 32) >> p.pw_log2);
            st_x = (quad * 32) & (pw - 1);
            box_live = st_y < p.P && st_x < p.Q;
        }
        bool waited = false;
        for (int pass = 0; pass < passes; ++pass) {
            const int col0 = (part * passes + pass) * cols;  // first tile column of this warp in this pass
            const int nw = tw.n_blk * BN + col0;             // ... as an output channel
            if (col0 >= BN) {
                // no columns for this warp in this pass: only keep step with the accumulator barriers
                if (!waited) {
                    if (!__all_sync(0xffffffffu, wait_bounded(&x.tmem_full[buf], buf_phase, x.abort_flag, 4))) return;
                    waited = true;
                }
                if (pass + 1 == passes) {
                    __syncwarp();
                    if (lane == 0) {
                        if (CG == 2) ptx::mbar_arrive_cluster_relaxed(ptx::mapa(ptx::smem_u32(&x.tmem_empty[buf]), 0));
                        else ptx::mbar_arrive_relaxed(&x.tmem_empty[buf]);
                    }
                }
                continue;
            }
            float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
            if (kScaled && nw + 4 * (lane & 15) < p.N) f = __ldg(reinterpret_cast<const float4 *>(fsrc + nw));
            int ent = 0;                                     // fused boundary: lane g fetches chunk g's slab entry
            if (MODE == kOutNextSlab && lane < 4 && nw + 16 * lane < p.N) ent = __ldg(p.next_ent + (nw >> 4) + lane);
            if (!waited) {
                PROF_T0(t0);
                const bool ok = wait_bounded(&x.tmem_full[buf], buf_phase, x.abort_flag, 4);
                PROF_ADD(prof_wait, t0);
                if (!__all_sync(0xffffffffu, ok)) return;
                ptx::tc_fence_after_sync();
                waited = true;
            }
            const uint32_t taddr = x.tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(SPLIT ? 2 * buf : buf) * x.buf_stride + (uint32_t)col0;
            PROF_T0(te0);
            uint32_t ra[32], rb[32];
            ptx::tmem_ld_32x32(taddr, ra);
            if (SPLIT) ptx::tmem_ld_32x32(taddr + x.buf_stride, rb);   // the other MMA warp's partial sums (32-column passes only)
            else if (cols == 64) ptx::tmem_ld_32x32(taddr + 32, rb);
            if (kScaled) {
                __syncwarp();                                      // the previous reads of the table are done
                reinterpret_cast<float4 *>(x.fac)[lane] = f;
                __syncwarp();
            }
            ptx::tmem_ld_wait();
            if (SPLIT) {
#pragma unroll
                for (int i = 0; i < 32; ++i) ra[i] += rb[i];
            }
            PROF_ADD(prof_ld, te0);
            PROF_T0(te1);
            if (pass + 1 == passes) {
                // the accumulator slice is in registers: hand it back to the MMA warp before the math
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    if (CG == 2) ptx::mbar_arrive_cluster_relaxed(ptx::mapa(ptx::smem_u32(&x.tmem_empty[buf]), 0));
                    else ptx::mbar_arrive_relaxed(&x.tmem_empty[buf]);
                }
            }
            int ents[4] = {0, 0, 0, 0};
            if (MODE == kOutNextSlab) {
#pragma unroll
                for (int g = 0; g < 4; ++g) ents[g] = __shfl_sync(0xffffffffu, ent, g);
            }
            if ((MODE == FLEXIQ_OUT_REQUANT_I8 || MODE == kOutNextSlab) && p.tma_store) {
                // Each warp stages 32 rows x 32 columns (1 KB, 32-byte swizzle: no bank conflicts) and one
                // lane hands them to a tiled bulk store, which writes whole sectors asynchronously and
                // drops the rows and columns that lie outside Y.
                const long long row0 = kPatch ? (box_live ? 0 : p.M) : row - lane;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t *r = h == 0 ? ra : rb;
                    const int n = nw + 32 * h;
                    if (32 * h < cols && n < p.N && row0 < p.M) {   // warp-uniform
                        const bool both = n + 16 < p.N;  // a 32-column box, else (last 16 channels of N) a 16-column one
                        uint32_t w[8];
                        if (MODE == kOutNextSlab) {
                            // the producer already emits the next layer's slab order: chunk c stays chunk c and
                            // is lowered when it lies below the next layer's max_4bit_ch
#pragma unroll
                            for (int g = 0; g < 2; ++g)
                                if (g == 0 || both) next_slab16(p, ents[2 * h + g], r + 16 * g, x.fac + 32 * h + 16 * g, x.fac + 64 + 32 * h + 16 * g, w + 4 * g);
                        } else {
                            finish16<FLEXIQ_OUT_REQUANT_I8>(r, x.fac + 32 * h, x.fac + 64 + 32 * h, w);
                            if (both) finish16<FLEXIQ_OUT_REQUANT_I8>(r + 16, x.fac + 32 * h + 16, x.fac + 64 + 32 * h + 16, w + 4);
                        }
                        if (lane == 0) ptx::bulk_wait_read_all();    // the previous store has read the buffer
                        __syncwarp();
                        if (both) {
                            const uint32_t dst = x.store_stage + (uint32_t)lane * 32u;
                            const uint32_t sw16 = ((uint32_t)lane >> 2 & 1u) << 4;
                            ptx::st_shared_128(dst + sw16, w[0], w[1], w[2], w[3]);
                            ptx::st_shared_128(dst + (sw16 ^ 16u), w[4], w[5], w[6], w[7]);
                        } else {
                            ptx::st_shared_128(x.store_stage + (uint32_t)lane * 16u, w[0], w[1], w[2], w[3]);
                        }
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            if (kPatch) ptx::tma_store_4d(both ? x.map_y : x.map_y16, x.store_stage, n, st_x, st_y, st_n);
                            else ptx::tma_store_2d(both ? x.map_y : x.map_y16, x.store_stage, n, (int)row0);
                            ptx::bulk_commit_group();
                        }
                    }
                }
            } else if (kHalf && p.tma_store) {
                // 16-bit outputs: 32 rows x 16 columns (32 bytes per row: the same 1 KB swizzled box) per store
                const long long row0 = kPatch ? (box_live ? 0 : p.M) : row - lane;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t *r = h == 0 ? ra : rb;
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        const int n = nw + 32 * h + 16 * g;
                        if (32 * h < cols && n < p.N && row0 < p.M) {   // warp-uniform
                            uint32_t w[16], hw[8];
                            finish16<FLEXIQ_OUT_DEQUANT_F32>(r + 16 * g, x.fac + 32 * h + 16 * g, x.fac + 64 + 32 * h + 16 * g, w);
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                hw[q] = pack2_f16<MODE == FLEXIQ_OUT_DEQUANT_BF16>(__uint_as_float(w[2 * q]), __uint_as_float(w[2 * q + 1]));
                            if (lane == 0) ptx::bulk_wait_read_all();    // the previous store has read the buffer
                            __syncwarp();
                            const uint32_t dst = x.store_stage + (uint32_t)lane * 32u;
                            const uint32_t sw16 = ((uint32_t)lane >> 2 & 1u) << 4;
                            ptx::st_shared_128(dst + sw16, hw[0], hw[1], hw[2], hw[3]);
                            ptx::st_shared_128(dst + (sw16 ^ 16u), hw[4], hw[5], hw[6], hw[7]);
                            ptx::fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) {
                                if (kPatch) ptx::tma_store_4d(x.map_y, x.store_stage, 2 * n, st_x, st_y, st_n);
                                else ptx::tma_store_2d(x.map_y, x.store_stage, 2 * n, (int)row0);
                                ptx::bulk_commit_group();
                            }
                        }
                    }
                }
            } else if (kElem == 4 && p.tma_store) {
                // 4-byte outputs: 32 rows x 8 columns per store (the same 32-byte rows)
                const long long row0 = kPatch ? (box_live ? 0 : p.M) : row - lane;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t *r = h == 0 ? ra : rb;
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        const int n = nw + 32 * h + 16 * g;
                        if (32 * h < cols && n < p.N && row0 < p.M) {   // warp-uniform
                            uint32_t w[16];
                            finish16<MODE>(r + 16 * g, x.fac + 32 * h + 16 * g, x.fac + 64 + 32 * h + 16 * g, w);
                            const uint32_t dst = x.store_stage + (uint32_t)lane * 32u;
                            const uint32_t sw16 = ((uint32_t)lane >> 2 & 1u) << 4;
#pragma unroll
                            for (int b = 0; b < 2; ++b) {
                                if (lane == 0) ptx::bulk_wait_read_all();
                                __syncwarp();
                                ptx::st_shared_128(dst + sw16, w[8 * b], w[8 * b + 1], w[8 * b + 2], w[8 * b + 3]);
                                ptx::st_shared_128(dst + (sw16 ^ 16u), w[8 * b + 4], w[8 * b + 5], w[8 * b + 6], w[8 * b + 7]);
                                ptx::fence_proxy_async_smem();
                                __syncwarp();
                                if (lane == 0) {
                                    if (kPatch) ptx::tma_store_4d(x.map_y, x.store_stage, 4 * (n + 8 * b), st_x, st_y, st_n);
                                    else ptx::tma_store_2d(x.map_y, x.store_stage, 4 * (n + 8 * b), (int)row0);
                                    ptx::bulk_commit_group();
                                }
                            }
                        }
                    }
                }
            } else
            if (row < p.M) {
                uint8_t *yrow = static_cast<uint8_t *>(p.Y) + (row * p.N + nw) * kElem;
#pragma unroll
                for (int h = 0; h < 2; ++h) {                       // two halves of 32 columns
                    const uint32_t *r = h == 0 ? ra : rb;
                    const int n = nw + 32 * h;
                    if (32 * h < cols && n < p.N) {
                        const bool second = n + 16 < p.N;  // columns 16..31 of this half are live
                        if (MODE == kOutNextSlab) {
                            // each 16-channel chunk goes to its place in the next layer's slab row
                            uint32_t w[8];
                            int pos[2] = {0, 0};
#pragma unroll
                            for (int g = 0; g < 2; ++g) {
                                if (g == 0 || second) {
                                    pos[g] = ents[2 * h + g] & 0xffffff;
                                    next_slab16(p, ents[2 * h + g], r + 16 * g, x.fac + 32 * h + 16 * g, x.fac + 64 + 32 * h + 16 * g, w + 4 * g);
                                }
                            }
                            uint8_t *srow = static_cast<uint8_t *>(p.Y) + row * p.N;
                            if (second && wide && pos[1] == pos[0] + 1 && (pos[0] & 1) == 0) st_global_256(srow + pos[0] * 16, w);
                            else {
                                st_global_128(srow + pos[0] * 16, w[0], w[1], w[2], w[3]);
                                if (second) st_global_128(srow + pos[1] * 16, w[4], w[5], w[6], w[7]);
                            }
                        } else if (MODE == FLEXIQ_OUT_REQUANT_I8) {
                            uint32_t w[8];
                            finish16<MODE>(r, x.fac + 32 * h, x.fac + 64 + 32 * h, w);
                            if (second) finish16<MODE>(r + 16, x.fac + 32 * h + 16, x.fac + 64 + 32 * h + 16, w + 4);
                            if (second && wide && ((nw & 31) == 0)) st_global_256(yrow + 32 * h, w);  // 32-byte aligned only then
                            else {
                                st_global_128(yrow + 32 * h, w[0], w[1], w[2], w[3]);
                                if (second) st_global_128(yrow + 32 * h + 16, w[4], w[5], w[6], w[7]);
                            }
                        } else if (kHalf) {
                            // 16-bit floating-point outputs: the fp32 result of the fma, rounded once more (to nearest even)
#pragma unroll
                            for (int g = 0; g < 2; ++g) {
                                if (g == 0 || second) {
                                    uint32_t w[16], hw[8];
                                    finish16<FLEXIQ_OUT_DEQUANT_F32>(r + 16 * g, x.fac + 32 * h + 16 * g, x.fac + 64 + 32 * h + 16 * g, w);
#pragma unroll
                                    for (int q = 0; q < 8; ++q)
                                        hw[q] = pack2_f16<MODE == FLEXIQ_OUT_DEQUANT_BF16>(__uint_as_float(w[2 * q]), __uint_as_float(w[2 * q + 1]));
                                    uint8_t *dst = yrow + (32 * h + 16 * g) * 2;
                                    if (y32) st_global_256(dst, hw);    // rows of 2-byte elements with N % 16 == 0 are 32-byte aligned
                                    else {
                                        st_global_128(dst, hw[0], hw[1], hw[2], hw[3]);
                                        st_global_128(dst + 16, hw[4], hw[5], hw[6], hw[7]);
                                    }
                                }
                            }
                        } else {
#pragma unroll
                            for (int g = 0; g < 2; ++g) {
                                if (g == 0 || second) {
                                    uint32_t w[16];
                                    finish16<MODE>(r + 16 * g, x.fac + 32 * h + 16 * g, x.fac + 64 + 32 * h + 16 * g, w);
                                    uint8_t *dst = yrow + (32 * h + 16 * g) * 4;
                                    if (y32) {                      // rows of 4-byte elements with N % 16 == 0 are 64-byte aligned
                                        st_global_256(dst, w);
                                        st_global_256(dst + 32, w + 8);
                                    } else {
#pragma unroll
                                        for (int q = 0; q < 4; ++q) st_global_128(dst + 16 * q, w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
                                    }
                                }
                            }
                        }
                    }
                }
            }
            PROF_ADD(prof_math, te1);
        }
        if (!kPatch && (buf ^= 1) == 0) buf_phase ^= 1;
    }
    if (p.tma_store && lane == 0) ptx::bulk_wait_all();  // the staged stores are performed
    if (quad == 2 && part == 0 && lane == 0) { PROF_STORE(8, prof_wait); PROF_STORE(9, clock64() - prof_start); PROF_STORE(10, prof_ld); PROF_STORE(11, prof_math); }
}

// CG = 1: one CTA per 128 x BN tile.  CG = 2: a CTA pair (cluster of two) per 256 x BN tile;
// each CTA loads its own 128 rows of A and its own half of B (no multicast), the leader
// CTA issues cta_group::2 MMAs that read both halves, and each CTA drains the 128
// accumulator rows held in its own TMEM.  Operand traffic from L2 per MAC drops by a third.
// PK = 1 (single CTA only): the low slab arrives as packed 4-bit tiles; eight expander warps
// widen them into the operand ring (eight epilogue warps remain).
// KIND 0: linear layers and 1x1 convolutions (plain 2-D copies, one K block per stage); KIND 1: everything a
// convolution may need (im2col copies, several taps per stage, resident weight tiles).  The issuing warps'
// instruction streams are on the critical path of a tile, so the first kind carries none of the second's code.
// SPLIT (tiles of at most 128 columns, one K block per stage, at least two stages per tile): the two MMA warps
// take the ring's stages in turn INSIDE a tile, each into an accumulator of its own, and the epilogue adds the
// two: for narrow MMAs (64 cycles each) the issuing warp's bookkeeping, not the pipe, bounds a K block, and two
// warps halve it.  No accumulator is shared, so no order between the warps' MMAs is needed; their waits on
// the ring stay in ring order (one hand-over phase per stage).
template <int CG, int PK, int KIND, bool SPLIT>
__global__ void __launch_bounds__(kThreads, 1)
mixed_gemm_kernel(const __grid_constant__ CUtensorMap mapA_lo, const __grid_constant__ CUtensorMap mapA_hi,
                  const __grid_constant__ CUtensorMap mapB_lo, const __grid_constant__ CUtensorMap mapB_hi,
                  const __grid_constant__ CUtensorMap mapB_st, const __grid_constant__ CUtensorMap mapY, const __grid_constant__ CUtensorMap mapY16,
                  const GemmParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    if (ptx::smem_u32(smem) & 1023u) {  // the swizzled operand tiles need 1024-byte alignment
        if (threadIdx.x == 0) atomicMax(&g_status_word, 0x200u);
        return;
    }
    uint8_t *stage_base = smem;
    uint8_t *factors = smem + kStageRegion;
    uint8_t *store_stage = factors + kNumWorkWarps * kFactorsPerWarp;  // 1024-byte aligned: the bulk stores' swizzle needs it
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(store_stage + kNumWorkWarps * kStoreStagePerWarp);
    uint64_t *empty_bar = full_bar + kMaxStages;
    uint64_t *tmem_full = empty_bar + kMaxStages;
    uint64_t *tmem_empty = tmem_full + 4;
    uint64_t *raw_full = tmem_empty + 4;
    uint64_t *raw_empty = raw_full + kRawStages;
    uint64_t *turn_bar = raw_empty + kRawStages;     // hand-over between the two MMA warps: one phase per tile
    uint32_t *tmem_ptr_s = reinterpret_cast<uint32_t *>(turn_bar + 1);
    constexpr int kEpiWarps = PK ? 8 : 16;
    constexpr int kExpWarps = PK ? 8 : 0;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_ptr_s + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int BN = p.BN;
    const bool k_im2col = KIND != 0 && p.im2col;      // compile-time false for KIND 0: the branches below fold away
    const int k_tps = KIND != 0 ? p.tps : 1;
    const bool k_bres = KIND != 0 && p.b_res;
    constexpr bool kPatch = KIND == 2;            // halo patch per tile, taps as row offsets (see GemmParams)
    const int b_rows = BN / CG;                       // rows of the B tile this CTA loads
    // one stage = tps sub-tiles of A (BM x BK each) followed by tps sub-tiles of B (b_rows x BK each)
    const int a_sub = BM * p.BK, b_sub = b_rows * p.BK, b_off = k_tps * a_sub;
    const int stage_bytes = kPatch ? p.patch_stage : (k_bres ? k_tps * a_sub : k_tps * (a_sub + b_sub));
    const int ring_off = k_bres ? ((p.T * b_sub + 1023) & ~1023) : 0;   // resident weight tiles lie in front of the ring
    const int num_tiles = p.m_tiles * p.n_tiles;
    const uint32_t cta_rank = CG == 2 ? ptx::cluster_ctarank() : 0u;
    const bool leader = cta_rank == 0;
    const int first_tile = blockIdx.x / CG, tile_step = gridDim.x / CG;
    // two accumulators (tiles in turn); SPLIT: two per tile, four in all
    const uint32_t buf_stride = BN <= 64 ? 64u : (BN <= 128 ? 128u : 256u);  // column offset from one accumulator to the next
    const uint32_t tmem_cols = ((SPLIT || kPatch) ? 4u : 2u) * buf_stride;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(&full_bar[s], PK ? kExpWarps : 1);  // packed path: every fill counts eight arrivals
            ptx::mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < 4; ++b) {
            ptx::mbar_init(&tmem_full[b], SPLIT ? 2 : 1);   // SPLIT: both MMA warps commit a tile
            // patch mode with 64-column tiles: half of the epilogue warps drain a tile (the others take the next one)
            ptx::mbar_init(&tmem_empty[b], (kPatch && BN == 64) ? kEpiWarps / 2 : CG * kEpiWarps);
        }
        for (int r = 0; r < kRawStages; ++r) {
            ptx::mbar_init(&raw_full[r], 1);
            ptx::mbar_init(&raw_empty[r], PK ? kExpWarps : 1);
        }
        ptx::mbar_init(turn_bar, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        if (CG == 2) { ptx::tmem_alloc_pair(tmem_ptr_s, tmem_cols); ptx::tmem_relinquish_pair(); }
        else { ptx::tmem_alloc(tmem_ptr_s, tmem_cols); ptx::tmem_relinquish(); }
    }
    ptx::tc_fence_before_sync();
    if (CG == 2) ptx::cluster_sync_all();  // the peer's barriers are initialised before anyone signals them
    else __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_s;
    // Everything above touched only this CTA's shared and tensor memory, so it may overlap the tail
    // of the previous kernel of the stream (programmatic dependent launch); wait for that kernel
    // (the prologue that writes the slabs) before reading or writing global memory.  This kernel
    // does not release its own successor early: a successor parked on the SMs slows the mainloop.
    ptx::pdl_wait();

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer
        // The whole warp walks the loops; one elected lane issues the copies.  K blocks run
        // low slab first (every tap, every channel block), then the high slab.
        if (ptx::elect_one()) {
            ptx::prefetch_tmap(&mapA_lo);
            ptx::prefetch_tmap(&mapA_hi);
            ptx::prefetch_tmap(&mapB_lo);
            ptx::prefetch_tmap(&mapB_hi);
            if (!PK && p.st_cb >= 0) ptx::prefetch_tmap(&mapB_st);
        }
        const uint32_t tx_bytes = (uint32_t)(CG * (BM * p.BK + b_rows * p.BK));  // both CTAs' loads
        const uint32_t stage0 = ptx::smem_u32(stage_base) + (uint32_t)ring_off;
        const uint32_t empty0 = ptx::smem_u32(empty_bar);
        const uint32_t full0 = ptx::smem_u32(full_bar);
        const uint32_t full0_lead = CG == 2 ? ptx::mapa(full0, 0) : full0;  // transaction bytes go to the leader's barrier
        uint32_t stage = 0, phase = 0;
        uint32_t rstage = 0, rphase = 0;                       // packed path: ring of raw 4-bit tiles
        const uint32_t raw0 = stage0 + (uint32_t)(p.stages * stage_bytes);
        const uint32_t raw_bytes = (uint32_t)((BM + BN) * (p.BK / 2));
        long long issued = 0;
        bool ok = true;
        PROF_DECL(prof_wait);
        PROF_T0(prof_start);
        TileWalk tw;
        tw.init(first_tile, tile_step, num_tiles, p.n_tiles);
        if (k_bres && tw.left > 0 && ptx::elect_one()) {
            // all taps' weight tiles of this CTA's (only) column block, once
            const uint32_t bar = ptx::smem_u32(&raw_full[0]);
            if (leader) ptx::mbar_expect_tx_s(bar, (uint32_t)(CG * p.T * b_sub));
            const uint32_t bar_lead = CG == 2 ? ptx::mapa(bar, 0) : bar;
            for (int t = 0; t < p.T; ++t)
                ptx::tma_load_2d_s<CG>(ptx::smem_u32(stage_base) + t * b_sub, &mapB_hi, bar_lead, t * p.b_tap_step, (int)cta_rank * b_rows);
        }
        __syncwarp();
        // Output pixel (image, row, column) of this CTA's first row in the current tile, kept up to date by
        // additions: the divisions are done once per kernel, not once per tile, in this single-lane loop.
        PixelWalk pw;
        if (k_im2col) pw.init(((long long)tw.m_blk * CG + cta_rank) * BM, (long long)tw.step_m * CG * BM, (long long)CG * BM, p.P, p.Q);
        int prev_m = tw.m_blk;
        for (; tw.left > 0 && ok; tw.next()) {
            const long long m0 = ((long long)tw.m_blk * CG + cta_rank) * BM;
            const int n0 = tw.n_blk * BN + (int)cta_rank * b_rows;
            int pix_w = 0, pix_h = 0, pix_n = 0;
            if (k_im2col) {
                if (tw.m_blk != prev_m) { pw.advance(tw.m_blk - prev_m - tw.step_m, p.P, p.Q); prev_m = tw.m_blk; }
                pix_n = pw.n;
                pix_h = pw.h * p.stride - p.pad;
                pix_w = pw.w * p.stride - p.pad;
            }
            if (kPatch) {
                // one copy per tile: TH + R - 1 input rows of PW pixels, starting one padding to the left of and above
                // the tile's first output pixel; what lies outside the image arrives as zeros
                PROF_T0(tq0);
                if (!__all_sync(0xffffffffu, wait_bounded(empty0 + 8 * stage, phase ^ 1, abort_flag, 1))) { ok = false; break; }
                PROF_ADD(prof_wait, tq0);
                if (ptx::elect_one()) {
                    const int img = tw.m_blk / p.tiles_per_img;
                    const int y0 = (tw.m_blk - img * p.tiles_per_img) * p.TH;
                    ptx::mbar_expect_tx_s(full0 + 8 * stage, (uint32_t)((p.patch_rows << p.pw_log2) * p.BK));
                    ptx::tma_load_4d_s(stage0 + stage * stage_bytes, &mapA_hi, full0 + 8 * stage, 0, -p.pad, y0 - p.pad, img);
                }
                __syncwarp();
                ++issued;
                if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                continue;
            }
            if (k_tps > 1) {
                // several filter taps per stage: one barrier round trip pays for all of them
                int tap_s = 0, tap_r = 0, tap_k = 0;   // running tap coordinates: no division in the issuing lane's loop
                for (int tap0 = 0; tap0 < p.T && ok; tap0 += k_tps) {
                    const int nt = min(k_tps, p.T - tap0);
                    PROF_T0(tq0);
                    if (!__all_sync(0xffffffffu, wait_bounded(empty0 + 8 * stage, phase ^ 1, abort_flag, 1))) { ok = false; break; }
                    PROF_ADD(prof_wait, tq0);
                    if (ptx::elect_one()) {
                        const uint32_t sa = stage0 + stage * stage_bytes;
                        if (leader) ptx::mbar_expect_tx_s(full0 + 8 * stage, (uint32_t)(CG * nt * (k_bres ? a_sub : a_sub + b_sub)));
                        const uint32_t bar = full0_lead + 8 * stage;
                        int ts = tap_s, tr = tap_r, tk = tap_k;
                        for (int i = 0; i < nt; ++i) {
                            ptx::tma_load_im2col_4d_s<CG>(sa + i * a_sub, &mapA_hi, bar, 0, pix_w, pix_h, pix_n, (uint16_t)ts, (uint16_t)tr);
                            if (!k_bres) ptx::tma_load_2d_s<CG>(sa + b_off + i * b_sub, &mapB_hi, bar, tk, n0);
                            tk += p.b_tap_step;
                            if (++ts == p.S) { ts = 0; ++tr; }
                        }
                    }
                    for (int i = 0; i < nt; ++i) {
                        tap_k += p.b_tap_step;
                        if (++tap_s == p.S) { tap_s = 0; ++tap_r; }
                    }
                    __syncwarp();
                    ++issued;
                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                }
                continue;
            }
            for (int part = 0; part < 2 && ok; ++part) {
                const int nb = part ? p.nb_hi : p.nb_lo;
                if (nb == 0) continue;
                const CUtensorMap *ma = part ? &mapA_hi : &mapA_lo;
                const CUtensorMap *mb = part ? &mapB_hi : &mapB_lo;
                // weights: slab-order [N][T*C]; the first run starts each tap at channel 0, the second at xb_hi0
                int xb_tap = part ? p.xb_hi0 : 0;
                int tap_r = 0, tap_s = 0;
                for (int tap = 0; tap < p.T && ok; ++tap) {
                    int xa = part ? p.xa_hi0 : 0, xb = xb_tap;
                    for (int cb = 0; cb < nb; ++cb) {
                        if (PK && part == 0) {
                            // packed low block: half-size raw tiles for the expander warps; the operand-ring
                            // stage this block will occupy is only counted here
                            if (!__all_sync(0xffffffffu, wait_bounded(&raw_empty[rstage], rphase ^ 1, abort_flag, 5))) { ok = false; break; }
                            if (ptx::elect_one()) {
                                const uint32_t ra = raw0 + rstage * raw_bytes;
                                const uint32_t bar = ptx::smem_u32(&raw_full[rstage]);
                                ptx::mbar_expect_tx_s(bar, raw_bytes);
                                if (k_im2col)
                                    ptx::tma_load_im2col_4d_s<1>(ra, ma, bar, xa >> 1, pix_w, pix_h, pix_n, (uint16_t)tap_s, (uint16_t)tap_r);
                                else
                                    ptx::tma_load_2d_s<1>(ra, ma, bar, xa >> 1, (int)m0);
                                ptx::tma_load_2d_s<1>(ra + BM * (p.BK / 2), mb, bar, xb >> 1, n0);
                            }
                            __syncwarp();
                            if (++rstage == kRawStages) { rstage = 0; rphase ^= 1; }
                            xa += p.BK;
                            xb += p.BK;
                            ++issued;
                            if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                            continue;
                        }
                        PROF_T0(t0);
                        if (!__all_sync(0xffffffffu, wait_bounded(empty0 + 8 * stage, phase ^ 1, abort_flag, 1))) { ok = false; break; }
                        PROF_ADD(prof_wait, t0);
                        if (ptx::elect_one()) {
                            const uint32_t sa = stage0 + stage * stage_bytes;
                            if (leader) ptx::mbar_expect_tx_s(full0 + 8 * stage, tx_bytes);
                            if (PK) ptx::mbar_arrive_count(&full_bar[stage], PK ? kExpWarps - 1 : 0);  // stand in for the expander warps
                            const uint32_t bar = full0_lead + 8 * stage;
                            if (k_im2col)
                                ptx::tma_load_im2col_4d_s<CG>(sa, ma, bar, xa, pix_w, pix_h, pix_n, (uint16_t)tap_s, (uint16_t)tap_r);
                            else
                                ptx::tma_load_2d_s<CG>(sa, ma, bar, xa, (int)m0);
                            // the block that max_4bit_ch falls into comes from the straddle buffer [N][T][BK]
                            if (!PK && part == 0 && cb == p.st_cb) ptx::tma_load_2d_s<CG>(sa + b_off, &mapB_st, bar, tap * p.BK, n0);
                            else ptx::tma_load_2d_s<CG>(sa + b_off, mb, bar, xb, n0);
                        }
                        __syncwarp();
                        xa += p.BK;
                        xb += p.BK;
                        ++issued;
                        if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                    }
                    xb_tap += p.C;
                    if (++tap_s == p.S) { tap_s = 0; ++tap_r; }
                }
            }
        }
        PROF_STORE(0, prof_wait);
        PROF_STORE(1, clock64() - prof_start);
        PROF_STORE(2, issued);
        if (!ok && lane == 0) {
            // drain: let the copies already in flight land before the CTA retires
            const int n_back = issued < p.stages ? (int)issued : p.stages;
            int s = (int)stage;
            uint32_t ph = phase;
            for (int i = 0; i < n_back; ++i) {
                if (--s < 0) { s = p.stages - 1; ph ^= 1; }
                for (uint32_t w = 0; w < (1u << 16); ++w) {
                    if (leader && ptx::mbar_try_wait(&full_bar[s], ph)) break;
                    __nanosleep(64);
                    if (!leader && w > 64) break;  // its loads credit the leader's barrier: give them a few microseconds
                }
            }
        }
    } else if (warp == 1 || (!PK && warp == 2 + kNumWorkWarps)) {
        // ------------------------------------------------------------- MMA issuers
        // The whole warp walks the loops; one elected lane issues the MMAs and their commits.
        // Two warps take the CTA's tiles in turn (even tiles and accumulator 0, odd tiles and accumulator 1;
        // on the packed path one warp takes them all): a lone warp shows the latency of every instruction, and
        // the bookkeeping of a tile boundary (≈ 500 cycles) then runs behind the other warp's MMAs.  The waits
        // on the ring stay in ring order: a warp starts on its tile's first stage only after the other has
        // passed the wait for its own last stage (one barrier phase per tile), so the parity of a ring barrier
        // means what it means to a single consumer.
        const bool duo = !PK;
        const int my = warp == 1 ? 0 : 1;
        if (leader) {
            const uint32_t idesc = ptx::idesc_i8(BM * CG, BN);
            const uint64_t adesc0 = ptx::smem_desc(ptx::smem_u32(stage_base) + (uint32_t)ring_off, p.BK);
            const uint32_t bres_lo = (uint32_t)ptx::smem_desc(ptx::smem_u32(stage_base), p.BK);   // resident weight tiles
            bool bres_ready = false;
            const uint32_t desc_hi = (uint32_t)(adesc0 >> 32);
            const uint32_t a_lo0 = (uint32_t)adesc0;
            const uint32_t b_lo0 = a_lo0 + (uint32_t)(b_off >> 4);
            const uint32_t stage_step = (uint32_t)(stage_bytes >> 4);  // stays inside the 14-bit address field
            const uint32_t empty0 = ptx::smem_u32(empty_bar);
            const uint32_t full0 = ptx::smem_u32(full_bar);
            const int ks_full = p.BK >> 5;
            uint32_t stage = 0, phase = 0;
            int buf = (duo && !SPLIT) ? my : 0;
            uint32_t buf_phase = 0;
            bool ok = true;
            PROF_DECL(prof_wait_acc);
            PROF_DECL(prof_wait_full);
            PROF_T0(prof_start);
            const int tile_slots = kPatch ? 1 : (k_tps > 1 ? (p.T + k_tps - 1) / k_tps : p.T * (p.nb_lo + p.nb_hi));  // ring stages per tile
            int ti = 0;                                          // index of the tile in this CTA's sequence
            TileWalk tw;
            for (tw.init(first_tile, tile_step, num_tiles, p.n_tiles); tw.left > 0 && ok; tw.next(), ++ti) {
                if (!SPLIT && duo && (ti & 1) != my) {
                    // the other warp's tile: step over its ring stages
                    stage += (uint32_t)tile_slots;
                    while (stage >= (uint32_t)p.stages) { stage -= (uint32_t)p.stages; phase ^= 1; }
                    continue;
                }
                int slot = 0;                                    // stages of this tile passed so far
                if (kPatch) { buf = ti & 3; buf_phase = (uint32_t)(ti >> 2) & 1u; }   // four accumulators, tile ti in ti mod 4
                PROF_T0(t0);
                if (!__all_sync(0xffffffffu, wait_bounded(&tmem_empty[buf], buf_phase ^ 1, abort_flag, 2))) break;
                PROF_ADD(prof_wait_acc, t0);
                // the other warp has passed the wait for the last stage of the tile before this one
                if (!SPLIT && duo && ti > 0 && !__all_sync(0xffffffffu, wait_bounded(turn_bar, (uint32_t)((ti - 1) & 1), abort_flag, 7))) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(SPLIT ? 2 * buf + my : buf) * buf_stride;
                const int g0 = ti * tile_slots;                  // SPLIT: number of this tile's first stage in the CTA's sequence
                uint32_t acc = 0;
                if (kPatch) {
                    const int ks = (p.C + 31) >> 5;  // K steps of one tap (C <= BK)
                    PROF_T0(tq1);
                    if (!__all_sync(0xffffffffu, wait_bounded(full0 + 8 * stage, phase, abort_flag, 3))) { ok = false; break; }
                    PROF_ADD(prof_wait_full, tq1);
                    if (lane == 0) ptx::mbar_arrive(turn_bar);   // the tile's only stage: the other warp may go on
                    if (!bres_ready) {
                        if (!__all_sync(0xffffffffu, wait_bounded(&raw_full[0], 0, abort_flag, 6))) { ok = false; break; }
                        bres_ready = true;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t a_lo = a_lo0 + stage * stage_step;
                    if (ptx::elect_one()) {
                        const uint32_t b_step = (uint32_t)(b_sub >> 4);
                        const uint32_t row16 = (uint32_t)(p.BK >> 4);              // one pixel row of the patch, in 16-byte units
                        uint32_t b_lo = bres_lo, a_row = a_lo;
                        const int R = p.T / p.S;
                        if (R == 3 && p.S == 3 && (ks == 2 || ks == 4)) {
                            // the usual case spelled out: the issuing lane's instruction stream bounds these small MMAs
                            const uint32_t down = row16 << p.pw_log2;
                            if (ks == 2) patch_taps_3x3<CG, 4, 2>(d_tmem, a_lo, down, b_lo, b_step, desc_hi, idesc);
                            else patch_taps_3x3<CG, 8, 4>(d_tmem, a_lo, down, b_lo, b_step, desc_hi, idesc);
                        } else
                        for (int r = 0; r < R; ++r) {
                            uint32_t a_tap = a_row;
                            for (int t = 0; t < p.S; ++t) {
                                if (ks == 2) {
                                    ptx::mma_i8_s<CG>(d_tmem, a_tap, b_lo, desc_hi, idesc, acc);
                                    ptx::mma_i8_s<CG>(d_tmem, a_tap + 2, b_lo + 2, desc_hi, idesc, 1);
                                } else if (ks == 4) {
                                    ptx::mma_i8_s<CG>(d_tmem, a_tap, b_lo, desc_hi, idesc, acc);
                                    ptx::mma_i8_s<CG>(d_tmem, a_tap + 2, b_lo + 2, desc_hi, idesc, 1);
                                    ptx::mma_i8_s<CG>(d_tmem, a_tap + 4, b_lo + 4, desc_hi, idesc, 1);
                                    ptx::mma_i8_s<CG>(d_tmem, a_tap + 6, b_lo + 6, desc_hi, idesc, 1);
                                } else {
                                    uint32_t a2 = acc;
                                    for (int k = 0; k < ks; ++k) { ptx::mma_i8_s<CG>(d_tmem, a_tap + 2 * k, b_lo + 2 * k, desc_hi, idesc, a2); a2 = 1; }
                                }
                                acc = 1;
                                a_tap += row16;                                    // next tap of the filter row: one pixel to the right
                                b_lo += b_step;
                            }
                            a_row += row16 << p.pw_log2;                           // next filter row: one patch row down
                        }
                        ptx::mma_commit_s<CG>(empty0 + 8 * stage);
                    }
                    __syncwarp();
                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                } else
                if (k_tps > 1) {
                    const int ks = (p.C + 31) >> 5;  // K steps of one tap (C <= BK)
                    for (int tap0 = 0; tap0 < p.T && ok; tap0 += k_tps) {
                        const int nt = min(k_tps, p.T - tap0);
                        PROF_T0(tq1);
                        if (!__all_sync(0xffffffffu, wait_bounded(full0 + 8 * stage, phase, abort_flag, 3))) { ok = false; break; }
                        PROF_ADD(prof_wait_full, tq1);
                        if (duo && ++slot == tile_slots && lane == 0) ptx::mbar_arrive(turn_bar);   // the other warp may go on
                        if (k_bres && !bres_ready) {
                            if (!__all_sync(0xffffffffu, wait_bounded(&raw_full[0], 0, abort_flag, 6))) { ok = false; break; }
                            bres_ready = true;
                        }
                        const uint32_t a_lo = a_lo0 + stage * stage_step;
                        const uint32_t b_lo = k_bres ? bres_lo + (uint32_t)tap0 * (uint32_t)(b_sub >> 4) : b_lo0 + stage * stage_step;
                        if (ptx::elect_one()) {
                            const uint32_t a_step = (uint32_t)(a_sub >> 4), b_step = (uint32_t)(b_sub >> 4);
                            if (nt == 3 && ks == 2) {
                                // three taps of 64 channels (a filter row of the 64-channel 3x3 convolutions): the issuing
                                // lane's instruction stream bounds these small MMAs, so no loop around them
                                ptx::mma_i8_s<CG>(d_tmem, a_lo, b_lo, desc_hi, idesc, acc);
                                ptx::mma_i8_s<CG>(d_tmem, a_lo + 2, b_lo + 2, desc_hi, idesc, 1);
                                ptx::mma_i8_s<CG>(d_tmem, a_lo + a_step, b_lo + b_step, desc_hi, idesc, 1);
                                ptx::mma_i8_s<CG>(d_tmem, a_lo + a_step + 2, b_lo + b_step + 2, desc_hi, idesc, 1);
                                ptx::mma_i8_s<CG>(d_tmem, a_lo + 2 * a_step, b_lo + 2 * b_step, desc_hi, idesc, 1);
                                ptx::mma_i8_s<CG>(d_tmem, a_lo + 2 * a_step + 2, b_lo + 2 * b_step + 2, desc_hi, idesc, 1);
                            } else {
                                uint32_t a2 = acc;
                                for (int i = 0; i < nt; ++i)
                                    for (int k = 0; k < ks; ++k) {
                                        ptx::mma_i8_s<CG>(d_tmem, a_lo + i * a_step + 2 * k, b_lo + i * b_step + 2 * k, desc_hi, idesc, a2);
                                        a2 = 1;
                                    }
                            }
                            ptx::mma_commit_s<CG>(empty0 + 8 * stage);
                        }
                        __syncwarp();
                        acc = 1;
                        if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                    }
                }
                for (int part = 0; part < 2 && ok && k_tps == 1 && !kPatch; ++part) {
                    const int nb = part ? p.nb_hi : p.nb_lo;
                    if (nb == 0) continue;
                    const int ks_last = part ? p.ks_last_hi : p.ks_last_lo;
                    for (int tap = 0; tap < p.T && ok; ++tap) {
                        for (int cb = 0; cb < nb; ++cb) {
                            if (SPLIT) {
                                const int g = g0 + slot;
                                if ((g & 1) != my) {   // the other warp's stage
                                    ++slot;
                                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                                    continue;
                                }
                                // the other warp has passed its wait for the stage before this one
                                if (g > 0 && !__all_sync(0xffffffffu, wait_bounded(turn_bar, (uint32_t)((g - 1) & 1), abort_flag, 7))) { ok = false; break; }
                            }
                            PROF_T0(t1);
                            if (!__all_sync(0xffffffffu, wait_bounded(full0 + 8 * stage, phase, abort_flag, 3))) { ok = false; break; }
                            PROF_ADD(prof_wait_full, t1);
                            if (SPLIT) { ++slot; if (lane == 0) ptx::mbar_arrive(turn_bar); }
                            else if (duo && ++slot == tile_slots && lane == 0) ptx::mbar_arrive(turn_bar);   // the other warp may go on
                            const uint32_t a_lo = a_lo0 + stage * stage_step, b_lo = b_lo0 + stage * stage_step;
                            const int ks = cb == nb - 1 ? ks_last : ks_full;
                            if (ptx::elect_one()) {
                                // 32 bytes of K per instruction: the descriptor address advances by 2 (16-byte units)
                                if (ks == 4) {
                                    ptx::mma_i8_s<CG>(d_tmem, a_lo, b_lo, desc_hi, idesc, acc);
                                    ptx::mma_i8_s<CG>(d_tmem, a_lo + 2, b_lo + 2, desc_hi, idesc, 1);
                                    ptx::mma_i8_s<CG>(d_tmem, a_lo + 4, b_lo + 4, desc_hi, idesc, 1);
                                    ptx::mma_i8_s<CG>(d_tmem, a_lo + 6, b_lo + 6, desc_hi, idesc, 1);
                                } else {
                                    uint32_t a2 = acc;
                                    for (int k = 0; k < ks; ++k) {
                                        ptx::mma_i8_s<CG>(d_tmem, a_lo + 2 * k, b_lo + 2 * k, desc_hi, idesc, a2);
                                        a2 = 1;
                                    }
                                }
                                ptx::mma_commit_s<CG>(empty0 + 8 * stage);  // frees the stage (in both CTAs of a pair)
                            }
                            __syncwarp();
                            acc = 1;
                            if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                        }
                    }
                }
                if (ok && ptx::elect_one()) ptx::mma_commit_s<CG>(ptx::smem_u32(&tmem_full[buf]));
                __syncwarp();
                if (kPatch) {}                                   // set from ti at the top of the loop
                else if (duo && !SPLIT) buf_phase ^= 1;          // this warp's accumulator again at its next tile
                else if ((buf ^= 1) == 0) buf_phase ^= 1;        // SPLIT: buf counts the tile's pair of accumulators
            }
            if (my == 0) {
            PROF_STORE(4, prof_wait_acc);
            PROF_STORE(5, prof_wait_full);
            PROF_STORE(6, clock64() - prof_start);
            }
        }
    } else {
        if (warp < 2 + kEpiWarps) {
            // --------------------------------------------------------- epilogue
            // warp e owns TMEM lane quadrant (warp & 3) and one column part of the tile;
            // the warps do not synchronise with one another.
            const int e = warp - 2;
            EpilogueCtx x;
            x.tmem_base = tmem_base; x.buf_stride = buf_stride; x.cta_rank = cta_rank;
            x.tmem_full = tmem_full; x.tmem_empty = tmem_empty; x.abort_flag = abort_flag;
            x.fac = reinterpret_cast<float *>(factors + e * kFactorsPerWarp);  // alpha[64] | beta[64]
            x.store_stage = ptx::smem_u32(store_stage + e * kStoreStagePerWarp);
            x.map_y = &mapY; x.map_y16 = &mapY16;
            x.first_tile = first_tile; x.tile_step = tile_step; x.num_tiles = num_tiles;
            x.parts = kEpiWarps / 4; x.arrivals_on = 1;
            if (p.out_mode == FLEXIQ_OUT_REQUANT_I8) epilogue_role<CG, FLEXIQ_OUT_REQUANT_I8, SPLIT, KIND>(p, x, warp & 3, e >> 2, lane);
            else if (p.out_mode == FLEXIQ_OUT_DEQUANT_F32) epilogue_role<CG, FLEXIQ_OUT_DEQUANT_F32, SPLIT, KIND>(p, x, warp & 3, e >> 2, lane);
            else if (p.out_mode == kOutNextSlab) epilogue_role<CG, kOutNextSlab, SPLIT, KIND>(p, x, warp & 3, e >> 2, lane);
            else if (p.out_mode == FLEXIQ_OUT_DEQUANT_F16) epilogue_role<CG, FLEXIQ_OUT_DEQUANT_F16, SPLIT, KIND>(p, x, warp & 3, e >> 2, lane);
            else if (p.out_mode == FLEXIQ_OUT_DEQUANT_BF16) epilogue_role<CG, FLEXIQ_OUT_DEQUANT_BF16, SPLIT, KIND>(p, x, warp & 3, e >> 2, lane);
            else epilogue_role<CG, FLEXIQ_OUT_ACC_I32, SPLIT, KIND>(p, x, warp & 3, e >> 2, lane);
        } else if (PK && warp < 2 + kNumWorkWarps) {
            // --------------------------------------------------------- expanders (packed path)
            // Widen each raw 4-bit tile into the operand ring: 8 packed bytes -> one 16-byte unit
            // (nibble << position) at its swizzled place, activations shifted by sx[group], weights
            // by sw[group][n].  Thread t owns weight row t of the tile and half of activation row
            // t mod 128; its positions for the coming K block are fetched before it waits for the
            // tile.  Walks the same K blocks as the producer and the MMA warp.
            const int tid_e = (warp - 2 - kEpiWarps) * 32 + lane;
            const int upr = p.BK >> 4;                    // 16-byte units per operand row: 8 or 4
            const int half = p.BK >> 1;                   // raw bytes per row: 64 or 32
            const int cpg_log2 = p.G == 16 ? 0 : (p.G == 32 ? 1 : 2);  // 16-channel chunks per group
            const bool raw_swz = half == 64;              // 64-byte raw rows are stored with the 64-byte swizzle
            uint8_t *raw_base = stage_base + p.stages * stage_bytes;
            const int raw_bytes = (BM + BN) * half;
            const int rowB = tid_e;                       // BN <= 256 = number of expander threads
            const bool hasB = rowB < BN;
            const int rowA = tid_e & (BM - 1);
            const int uA0 = (tid_e >> 7) * (upr >> 1);    // first activation unit of this thread
            uint32_t stage = 0, phase = 0, rstage = 0, rphase = 0;
            bool ok = true;
            PROF_DECL(prof_x_raw); PROF_DECL(prof_x_empty); PROF_DECL(prof_x_work); PROF_DECL(prof_x_fence);
            PROF_T0(prof_x_start);
            TileWalk tw;
            for (tw.init(first_tile, tile_step, num_tiles, p.n_tiles); tw.left > 0 && ok; tw.next()) {
                const int n0 = tw.n_blk * BN;
                const bool liveB = hasB && n0 + rowB < p.N;
                const int colB = liveB ? n0 + rowB : 0;      // a valid column of the position table for every thread
                for (int part = 0; part < 2 && ok; ++part) {
                    const int nb = part ? p.nb_hi : p.nb_lo;
                    for (int tap = 0; tap < p.T && ok; ++tap) {
                        // The positions of a K block's chunks come from global memory (the 221 KB of shared memory
                        // leave almost no L1, so every fetch goes to L2): those of block cb + 1 are requested before
                        // block cb is widened.  The requests are unconditional (clamped indices); what a thread does
                        // not own is zeroed when the values are taken over.
                        int nxB[8], nxA[4];
                        const int last_chunk = (p.C_lo >> 4) - 1;
                        auto request = [&](int cb) {
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const int chunk = min(cb * upr + (u < upr ? u : 0), last_chunk);
                                nxB[u] = __ldg(p.sw + (size_t)(chunk >> cpg_log2) * p.N + colB);
                            }
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const int chunk = min(cb * upr + uA0 + (k < (upr >> 1) ? k : 0), last_chunk);
                                nxA[k] = __ldg(p.sx + (chunk >> cpg_log2));
                            }
                        };
                        if (part == 0 && nb > 0) request(0);
                        for (int cb = 0; cb < nb; ++cb) {
                            if (part == 0) {
                                int shB[8], shA[4];
#pragma unroll
                                for (int u = 0; u < 8; ++u) shB[u] = (u < upr && liveB && (cb * upr + u) * 16 < p.C_lo) ? nxB[u] : 0;
#pragma unroll
                                for (int k = 0; k < 4; ++k) shA[k] = (k < (upr >> 1) && (cb * upr + uA0 + k) * 16 < p.C_lo) ? nxA[k] : 0;
                                if (cb + 1 < nb) request(cb + 1);
                                PROF_T0(tx0);
                                bool w1 = wait_bounded(&raw_full[rstage], rphase, abort_flag, 6);
                                PROF_ADD(prof_x_raw, tx0);
                                PROF_T0(tx1);
                                w1 = w1 && wait_bounded(&empty_bar[stage], phase ^ 1, abort_flag, 7);
                                PROF_ADD(prof_x_empty, tx1);
                                if (!__all_sync(0xffffffffu, w1)) { ok = false; break; }
                                PROF_T0(tx2);
                                const uint8_t *rawA = raw_base + rstage * raw_bytes;
                                const uint8_t *rawB = rawA + BM * half;
                                uint8_t *dstA = stage_base + stage * stage_bytes;
                                uint8_t *dstB = dstA + b_off;
                                if (hasB) {
                                    const uint8_t *src = rawB + rowB * half;
                                    uint8_t *dst = dstB + rowB * p.BK;
                                    const int xr = raw_swz ? ((rowB >> 1) & 3) : 0;
                                    const int xd = upr == 8 ? (rowB & 7) : ((rowB >> 1) & 3);
#pragma unroll
                                    for (int v = 0; v < 4; ++v) {             // 16 raw bytes = two units
                                        if (2 * v < upr) {
                                            const uint4 q = *reinterpret_cast<const uint4 *>(src + ((v ^ xr) << 4));
                                            uint32_t o[4];
                                            unpack16(q.x, q.y, shB[2 * v], o);
                                            *reinterpret_cast<uint4 *>(dst + (((2 * v) ^ xd) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                                            unpack16(q.z, q.w, shB[2 * v + 1], o);
                                            *reinterpret_cast<uint4 *>(dst + (((2 * v + 1) ^ xd) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                                        }
                                    }
                                }
                                {
                                    const uint8_t *src = rawA + rowA * half;
                                    uint8_t *dst = dstA + rowA * p.BK;
                                    const int xr = raw_swz ? ((rowA >> 1) & 3) : 0;
                                    const int xd = upr == 8 ? (rowA & 7) : ((rowA >> 1) & 3);
#pragma unroll
                                    for (int k = 0; k < 2; ++k) {             // this thread's half of the row
                                        if (2 * k < (upr >> 1)) {
                                            const int v = (uA0 >> 1) + k;
                                            const uint4 q = *reinterpret_cast<const uint4 *>(src + ((v ^ xr) << 4));
                                            uint32_t o[4];
                                            unpack16(q.x, q.y, shA[2 * k], o);
                                            *reinterpret_cast<uint4 *>(dst + (((2 * v) ^ xd) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                                            unpack16(q.z, q.w, shA[2 * k + 1], o);
                                            *reinterpret_cast<uint4 *>(dst + (((2 * v + 1) ^ xd) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                                        }
                                    }
                                }
                                PROF_ADD(prof_x_work, tx2);
                                PROF_T0(tx3);
                                ptx::fence_proxy_async_smem();  // generic-proxy writes become visible to the MMA's reads
                                __syncwarp();
                                PROF_ADD(prof_x_fence, tx3);
                                if (lane == 0) {
                                    ptx::mbar_arrive(&full_bar[stage]);
                                    ptx::mbar_arrive(&raw_empty[rstage]);
                                }
                                if (++rstage == kRawStages) { rstage = 0; rphase ^= 1; }
                            }
                            if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                        }
                    }
                }
            }
            if (tid_e == 0) { PROF_STORE(10, prof_x_raw); PROF_STORE(11, prof_x_empty); PROF_STORE(12, prof_x_work); PROF_STORE(13, prof_x_fence); PROF_STORE(14, clock64() - prof_x_start); }
        }
    }

    ptx::tc_fence_before_sync();
    if (CG == 2) ptx::cluster_sync_all();  // neither CTA frees TMEM or retires while its peer still works
    else __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        if (CG == 2) ptx::tmem_dealloc_pair(tmem_base, tmem_cols);
        else ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
}

// Per-output-channel factors of a call: REQUANT alpha = (S_x * S_w[n]) / S_y, beta = bias[n] / S_y;
// DEQUANT alpha = S_x * S_w[n], beta = bias[n].  Each operation rounds once, in fp32.
__global__ void scale_vectors_kernel(int N, float x_scale, float y_scale, int requant, const float *__restrict__ w_scale,
                                     const float *__restrict__ bias, float *__restrict__ alpha, float *__restrict__ beta)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    ptx::pdl_wait();  // the previous kernel of the stream may still read the table
    if (n >= N) return;
    const float sxw = __fmul_rn(x_scale, w_scale[n]);
    const float bv = bias ? bias[n] : 0.f;
    alpha[n] = requant ? __fdiv_rn(sxw, y_scale) : sxw;
    beta[n] = requant ? __fdiv_rn(bv, y_scale) : bv;
}

// Test hook: one warp waits, with the mainloop's own bounded wait but a limit of about a millisecond, on a barrier
// that nothing ever arrives on; a second barrier that IS arrived on shows the same routine returning at once.
__global__ void wait_expiry_kernel(int *result)
{
    __shared__ uint64_t bars[2];
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bars[0], 1);
        ptx::mbar_init(&bars[1], 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) ptx::mbar_arrive(&bars[1]);
    __syncwarp();
    const bool served = wait_slow(ptx::smem_u32(&bars[1]), 0, &abort_flag, 15, 1024u);    // completes: returns true
    const bool starved = wait_slow(ptx::smem_u32(&bars[0]), 0, &abort_flag, 15, 1024u);   // never completes: gives up
    if (threadIdx.x == 0) {
        result[0] = served ? 1 : 0;
        result[1] = starved ? 1 : 0;
        result[2] = abort_flag;
    }
}

// The straddle block of the masked path (straddle.cuh) for a GEMM that no prologue launch precedes.
__global__ void straddle_kernel(const StraddleJob job)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    ptx::pdl_wait();  // the previous kernel of the stream may still read the block
    if (idx < (long long)job.rows * (job.BK >> 4)) straddle_write_unit(job, idx);
}

// ------------------------------------------------------------------------------------
// host side

// Tile shape, from a cost model in SM cycles whose constants were fitted to measured times of every
// tile shape on twenty layer shapes (ViT-B, DeiT-S at batch 1 and 8, ResNet-50 convolutions):
//   per K block  max(MMA 2*BN cycles per 128 bytes of K;  TMA fill of (128 + BN/cg) rows at 90 bytes per
//                cycle, 70 when (almost) every SM is loading, and at least 3.5 cycles per 64-byte row;
//                a floor of 350 cycles, 500 with every SM busy)
//   per tile     the K blocks + 800 cycles; its epilogue (800 + 4*BN cycles) overlaps the next tile
//   in all       waves * tile + one epilogue that nothing overlaps + 1600 cycles for a CTA pair
//                (cluster launch and barriers), which pays off once the machine is full.
struct TileChoice { int cg, bn; };
static TileChoice g_forced_tile{0, 0};  // test hook: 0 = choose automatically
static TileChoice choose_tile(long long M, int N, int k_blocks, int bk, int sms)
{
    const int bns[4] = {256, 192, 128, 64};
    TileChoice best{1, 256};
    double best_cost = 1e300;
    for (int cg = 2; cg >= 1; --cg)  // ties go to pairs: they halve the B traffic per SM
        for (int i = 0; i < 4; ++i) {
            const int bn = bns[i];
            if (cg == 2 && bn < 128) continue;
            const long long m_tiles = (M + (long long)BM * cg - 1) / ((long long)BM * cg);
            const long long n_tiles = (N + bn - 1) / bn;
            const long long slots = sms / cg;
            const long long tiles = m_tiles * n_tiles;
            const long long waves = (tiles + slots - 1) / slots;
            const bool busy = (tiles < slots ? tiles : slots) * cg >= 140;
            const double rows = 128.0 + (double)bn / cg;
            const double mma = 2.0 * bn * bk / 128.0;
            double tma = rows * bk / (busy ? 70.0 : 90.0);
            if (bk == 64 && tma < rows * 3.5) tma = rows * 3.5;
            const double floor_kb = (busy ? 500.0 : 350.0) * (bk == 128 ? 1.0 : 0.6);
            double per_kb = mma > tma ? mma : tma;
            if (per_kb < floor_kb) per_kb = floor_kb;
            const double mainloop = k_blocks * per_kb + 800.0;
            const double epi = 800.0 + 4.0 * bn;
            const double cost = (double)waves * (mainloop > epi ? mainloop : epi) + epi + (cg == 2 ? 1600.0 : 0.0);
            if (cost < best_cost - 1e-9) { best_cost = cost; best = TileChoice{cg, bn}; }
        }
    return best;
}

static int make_map_im2col(CUtensorMap *map, const void *base, int Cpart, long long pitch, int Nb, int H, int W,
                           int R, int S, int stride, int pad, int bk, int swizzle_bytes)
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
                     swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE),
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return set_error(FLEXIQ_ERR_CUDA, "cuTensorMapEncodeIm2col failed with CUresult %d", (int)r);
    return FLEXIQ_OK;
}

// 4-D byte tensor map over an NHWC tensor: (row_bytes of channels, W, H, Nb), box (box_bytes, bx, by, 1).
static int make_map_nhwc(CUtensorMap *map, const void *base, uint64_t row_bytes, int W, int H, int Nb, uint32_t box_bytes,
                         uint32_t bx, uint32_t by, int swizzle_bytes)
{
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return set_error(FLEXIQ_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    if ((reinterpret_cast<uintptr_t>(base) & 15) != 0 || (row_bytes & 15) != 0)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "tensor base %p / pixel pitch %llu not 16-byte aligned", base, (unsigned long long)row_bytes);
    cuuint64_t dims[4] = {row_bytes, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)Nb};
    cuuint64_t strides[3] = {row_bytes, row_bytes * W, row_bytes * W * H};
    cuuint32_t box[4] = {box_bytes, bx, by, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUtensorMapSwizzle swz = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                 : (swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                 : (swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE));
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return set_error(FLEXIQ_ERR_CUDA, "cuTensorMapEncodeTiled (4-D) failed with CUresult %d (box %u x %u x %u)", (int)r, box_bytes, bx, by);
    return FLEXIQ_OK;
}

template <int CG, int PK, int KIND, bool SPLIT>
static int launch_kernel(const CUtensorMap &a_lo, const CUtensorMap &a_hi, const CUtensorMap &b_lo, const CUtensorMap &b_hi,
                         const CUtensorMap &b_st, const CUtensorMap &y_map, const CUtensorMap &y_map16, const GemmParams &p, int sms, cudaStream_t st)
{
    static bool attr_set[64] = {};   // per instantiation
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 64 && !attr_set[dev]) {
        FLEXIQ_CUDA_TRY(cudaFuncSetAttribute(mixed_gemm_kernel<CG, PK, KIND, SPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        attr_set[dev] = true;
    }
    const long long tiles = (long long)p.m_tiles * p.n_tiles;
    const long long slots = sms / CG;
    const unsigned grid = (unsigned)((tiles < slots ? tiles : slots) * CG);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // overlap this launch's preamble with the predecessor's tail
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    FLEXIQ_CUDA_TRY(cudaLaunchKernelEx(&cfg, mixed_gemm_kernel<CG, PK, KIND, SPLIT>, a_lo, a_hi, b_lo, b_hi, b_st, y_map, y_map16, p));
    return FLEXIQ_OK;
}

// Masked path: writes the straddle block for the current max_4bit_ch when the stream does not hold it yet
// (a prologue launch at this ratio normally has written it already).
static int sync_straddle(Layer *L, cudaStream_t st)
{
    if (!straddle_in_use(L) || !straddle_stale(L, st)) return FLEXIQ_OK;
    StraddleJob job{};
    job.wst = L->wst; job.w8m = L->w8m; job.w8 = L->w8;
    job.rows = L->N * L->R * L->S;
    job.C = L->C;
    job.BK = choose_bk(L);
    job.blk0 = (L->K_lo / job.BK) * job.BK;
    job.K_lo = L->K_lo;
    const long long total = (long long)job.rows * (job.BK >> 4);
    straddle_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(job);
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    straddle_written(L, st);
    return FLEXIQ_OK;
}

static int run_mixed(Layer *L, const uint8_t *X4, const int8_t *X8, const uint8_t *x_shift, long long M, int Nb, int H,
                     int W, float x_scale, float y_scale, int out_mode, void *Y, cudaStream_t st,
                     const Layer *next = nullptr, int relu = 0, int out_order = 0)
{
    if (next) {
        // fused layer boundary: Y is the next layer's masked slab, y_scale its activation scale
        if (next->lowbit_path != FLEXIQ_LOWBIT_MASKED_I8)
            return set_error(FLEXIQ_ERR_UNSUPPORTED, "the next layer must use the masked low-bit path");
        if (next->C != L->N)
            return set_error(FLEXIQ_ERR_INVALID_ARG, "next layer has %d input channels, this layer %d output channels", next->C, L->N);
        if (next->device != L->device) return set_error(FLEXIQ_ERR_INVALID_ARG, "the two layers live on different devices");
        if (out_order != FLEXIQ_ORDER_ORIGINAL && out_order != FLEXIQ_ORDER_NEXT_SLAB)
            return set_error(FLEXIQ_ERR_INVALID_ARG, "unknown out_order %d", out_order);
        out_mode = kOutNextSlab;
    } else if (out_mode != FLEXIQ_OUT_ACC_I32 && out_mode != FLEXIQ_OUT_REQUANT_I8 && out_mode != FLEXIQ_OUT_DEQUANT_F32 &&
               out_mode != FLEXIQ_OUT_DEQUANT_F16 && out_mode != FLEXIQ_OUT_DEQUANT_BF16)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "unknown out_mode %d", out_mode);
    if ((out_mode == FLEXIQ_OUT_REQUANT_I8 || next) && !(y_scale > 0.0f))
        return set_error(FLEXIQ_ERR_INVALID_ARG, "y_scale %g must be positive", (double)y_scale);
    if (M == 0) return FLEXIQ_OK;
    const int C_lo = L->K_lo, C_hi = L->C - C_lo;
    if (!Y) return set_error(FLEXIQ_ERR_INVALID_ARG, "Y_dev is NULL");
    const bool packed_path = L->lowbit_path == FLEXIQ_LOWBIT_PACKED_U4;
    if (!packed_path && !X4) return set_error(FLEXIQ_ERR_INVALID_ARG, "X4_dev is NULL: on the masked path it is the whole slab");
    if (packed_path && C_lo > 0 && !X4) return set_error(FLEXIQ_ERR_INVALID_ARG, "X4_dev is NULL but K_lo = %d", C_lo);
    if (packed_path && C_hi > 0 && !X8) return set_error(FLEXIQ_ERR_INVALID_ARG, "X8_dev is NULL but K_hi = %d", C_hi);
    if ((reinterpret_cast<uintptr_t>(Y) | reinterpret_cast<uintptr_t>(X4) | (packed_path ? reinterpret_cast<uintptr_t>(X8) : 0)) & 15)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "X4_dev, X8_dev and Y_dev must be 16-byte aligned");
    const bool packed = L->lowbit_path == FLEXIQ_LOWBIT_PACKED_U4 && C_lo > 0;
    if (packed && L->is_conv && (L->C % 32) != 0)
        return set_error(FLEXIQ_ERR_UNSUPPORTED, "packed low-bit convolution needs Cin %% 32 == 0 (TMA start alignment of the 4-bit weight taps)");
    int rc = check_device_sm100();
    if (rc) return rc;
    if ((rc = check_layer_device(L))) return rc;
    // the slabs must have been written at the ratio now in force (known buffers only)
    if (packed_path) {
        if (C_lo > 0 && (rc = check_slab(L, X4, "X4_dev"))) return rc;
        if (C_hi > 0 && (rc = check_slab(L, X8, "X8_dev"))) return rc;
    } else if ((rc = check_slab(L, X4, "X4_dev"))) return rc;
    const int sms = device_sm_count(L->device);

    GemmParams p{};
    p.M = M; p.N = L->N; p.C = L->C; p.C_lo = packed ? C_lo : 0; p.C_hi = packed ? C_hi : L->C;
    p.T = L->R * L->S; p.S = L->S;
    p.BK = choose_bk(L);
    p.st_cb = -1;
    p.b_tap_step = L->C;
    int b_whole = 0;   // masked multi-tap stages: 0 = w8, 1 = w8m, 2 = straddle buffer
    if (packed) {
        p.nb_lo = (p.C_lo + p.BK - 1) / p.BK;
        p.nb_hi = (p.C_hi + p.BK - 1) / p.BK;
        p.ks_last_lo = (p.C_lo - (p.nb_lo - 1) * p.BK + 31) >> 5;
        p.ks_last_hi = (p.C_hi - (p.nb_hi - 1) * p.BK + 31) >> 5;
        p.xa_hi0 = 0;          // the 8-bit groups have a slab of their own
        p.xb_hi0 = C_lo;
    } else {
        // Masked path: activations are one slab [rows][C], and the mainloop is a plain 8-bit GEMM over whole
        // K blocks whatever the ratio: blocks below max_4bit_ch read w8m, blocks above it w8, and the block
        // the boundary falls into (if any) the straddle buffer.  Nothing else depends on the ratio.
        const int nbt = (L->C + p.BK - 1) / p.BK;
        const bool st_blk = straddle_in_use(L);
        if ((rc = sync_straddle(L, st))) return rc;
        p.nb_lo = C_lo / p.BK + (st_blk ? 1 : 0);
        if (C_lo == L->C) p.nb_lo = nbt;
        p.nb_hi = nbt - p.nb_lo;
        if (st_blk) p.st_cb = p.nb_lo - 1;
        const int ks_end = (L->C - (nbt - 1) * p.BK + 31) >> 5;   // the last block of a tap may be partial
        p.ks_last_lo = p.nb_hi == 0 ? ks_end : p.BK >> 5;
        p.ks_last_hi = ks_end;
        p.xa_hi0 = p.xb_hi0 = p.nb_lo * p.BK;
        b_whole = C_lo == 0 ? 0 : (C_lo == L->C ? 1 : 2);   // when one K block holds all channels
    }
    p.im2col = L->is_conv && (L->R != 1 || L->S != 1 || L->stride != 1 || L->pad != 0);
    p.stride = L->stride; p.pad = L->pad;
    if (L->is_conv) {
        p.P = (H + 2 * L->pad - L->R) / L->stride + 1;
        p.Q = (W + 2 * L->pad - L->S) / L->stride + 1;
    }
    p.out_mode = out_mode; p.Y = Y;
    if (next) { p.next_ent = out_order == FLEXIQ_ORDER_NEXT_SLAB ? next->chunk_ent_slab : next->chunk_ent; p.next_K_lo = next->K_lo; p.relu = relu != 0; }
    // The per-output-channel factors depend on the call's scales.  The handle keeps a few factor tables, each
    // written once for one (kind, S_x, S_y) and never changed while anything may still depend on it, so a
    // table that a captured graph reads (or writes) stays what that graph expects whatever runs in between.
    // The fused boundary re-quantizes with the REQUANT factors; the three floating-point outputs share theirs.
    const int fmode = next ? FLEXIQ_OUT_REQUANT_I8
                           : ((out_mode == FLEXIQ_OUT_DEQUANT_F16 || out_mode == FLEXIQ_OUT_DEQUANT_BF16) ? FLEXIQ_OUT_DEQUANT_F32 : out_mode);
    if (fmode != FLEXIQ_OUT_ACC_I32) {
        const unsigned long long cap = stream_capture_id(st);
        const float ys_key = fmode == FLEXIQ_OUT_REQUANT_I8 ? y_scale : 0.0f;
        Layer::FactorTable *ft = nullptr;
        for (int i = 0; i < Layer::kFactorTables && !ft; ++i)
            if (L->factors[i].keyed && L->factors[i].mode == fmode && L->factors[i].xs == x_scale && L->factors[i].ys == ys_key) ft = &L->factors[i];
        if (!ft) {
            // a table nothing captured depends on, taken in turn; failing that the scratch table, rewritten by every call
            for (int k = 0; k < Layer::kFactorTables && !ft; ++k) {
                Layer::FactorTable *c = &L->factors[(L->factor_next + k) % Layer::kFactorTables];
                if (!c->pinned) { ft = c; L->factor_next = (int)(c - L->factors + 1) % Layer::kFactorTables; }
            }
            if (!ft) ft = &L->factors[Layer::kFactorTables];
            ft->mode = fmode; ft->xs = x_scale; ft->ys = ys_key;
            ft->keyed = ft != &L->factors[Layer::kFactorTables];   // the scratch table is never found again
            ft->on_device = 0; ft->cap_id = 0;
        }
        // The values are on the device for this call when an eager call wrote them (they then stay: a keyed table is
        // only ever rewritten with the same values) or when this very capture already holds the write.  A write that
        // only another captured graph holds does not count: that graph may never have run.
        if (!(ft->on_device || (cap && ft->cap_id == cap))) {
            scale_vectors_kernel<<<(L->N + 255) / 256, 256, 0, st>>>(L->N, x_scale, y_scale, fmode == FLEXIQ_OUT_REQUANT_I8,
                                                                     L->w_scale, L->bias, ft->alpha, ft->beta);
            FLEXIQ_CUDA_TRY(cudaGetLastError());
            if (cap) ft->cap_id = cap;
            else ft->on_device = ft->keyed;
        }
        if (cap && ft->keyed) ft->pinned = 1;   // a graph now reads (or rewrites) this table with these values
        p.alpha = ft->alpha; p.beta = ft->beta;
    }
    TileChoice tc = g_forced_tile.cg ? g_forced_tile : choose_tile(M, L->N, p.T * (p.nb_lo + p.nb_hi), p.BK, sms);
    if (packed && tc.cg == 2) {  // the packed path runs single CTAs: re-choose among those
        tc.cg = 1;
        if (!g_forced_tile.cg) {
            const long long mt = (M + BM - 1) / BM;
            tc.bn = 256;
            long long best = -1;
            const int bns[4] = {256, 192, 128, 64};
            for (int i = 0; i < 4; ++i) {
                // the expander warps widen the tile's 128 + BN rows for every K block: that, not the MMAs, is a tile's time
                const long long tiles = mt * ((L->N + bns[i] - 1) / bns[i]);
                const long long cost = ((tiles + sms - 1) / sms) * (BM + bns[i]);
                if (best < 0 || cost < best) { best = cost; tc.bn = bns[i]; }
            }
        }
    }
    // Patch mode (see GemmParams): stride-1 filters of more than one tap whose channels fit one K block and whose
    // output channels fit one tile, the weights of all taps resident in shared memory.
    bool patch = false;
    int patch_pw = 8;
    if (!packed && !g_forced_tile.cg && p.im2col && L->stride == 1 && L->C <= p.BK && L->N <= 128 && W + L->pad <= 128) {
        while (patch_pw < W + L->pad) patch_pw *= 2;
        const int th = BM / patch_pw, bn_p = L->N <= 64 ? 64 : 128;
        const int rows = th + L->R - 1 + (W + 2 * L->pad > patch_pw ? 1 : 0);
        const int stage = ((rows * patch_pw * p.BK) + 1023) & ~1023;
        const int b_all = ((p.T * bn_p * p.BK) + 1023) & ~1023;
        if (b_all + 2 * stage <= kStageRegion && rows <= 256) {
            patch = true;
            tc.cg = 1; tc.bn = bn_p;
            p.TH = th; p.patch_stage = stage; p.patch_rows = rows;
            p.pw_log2 = 0;
            while ((1 << p.pw_log2) < patch_pw) ++p.pw_log2;
            p.tiles_per_img = (p.P + th - 1) / th;
        }
    }
    const int bn = tc.bn, cg = tc.cg;
    p.sx = x_shift ? x_shift : L->sx;
    p.sw = L->sw;
    p.G = L->G;
    p.m_tiles = patch ? Nb * p.tiles_per_img : (int)((M + (long long)BM * cg - 1) / ((long long)BM * cg));
    p.BN = bn;
    p.n_tiles = (L->N + bn - 1) / bn;
    p.tps = 1;
    if (!packed && !patch && p.im2col && L->C <= p.BK && L->S > 1) {
        // convolution whose channels fit one K block: a stage holds up to a filter row of taps
        const int per_tap = (BM + bn / cg) * p.BK;
        const int limit = 49152 / per_tap;
        p.tps = L->S < limit ? L->S : limit;
        if (p.tps < 1) p.tps = 1;
    }
    p.stages = kStageRegion / (p.tps * (BM + bn / cg) * p.BK);
    if (p.tps > 1 && p.n_tiles == 1) {
        const int b_all = ((p.T * (bn / cg) * p.BK + 1023) / 1024) * 1024;
        const int st = (kStageRegion - b_all) / (p.tps * BM * p.BK);
        if (b_all <= 65536 && st >= 4) { p.b_res = 1; p.stages = st; }
    }
    if (patch) {
        p.b_res = 1;
        p.stages = (kStageRegion - (((p.T * bn * p.BK) + 1023) & ~1023)) / p.patch_stage;
    }
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    if (packed) {  // room for the ring of raw 4-bit tiles behind the operand ring
        const int raw = kRawStages * (BM + bn) * (p.BK / 2);
        p.stages = (kStageRegion - raw) / ((BM + bn) * p.BK);
        if (p.stages > kMaxStages) p.stages = kMaxStages;
    }
    // activation maps (per call: they depend on the caller's buffers, M and the ratio);
    // an empty slab borrows the other one's map and is never addressed
    CUtensorMap a_lo, a_hi;
    const bool half_out = out_mode == FLEXIQ_OUT_DEQUANT_F16 || out_mode == FLEXIQ_OUT_DEQUANT_BF16;
    const bool word_out = out_mode == FLEXIQ_OUT_DEQUANT_F32 || out_mode == FLEXIQ_OUT_ACC_I32;
    const int y_elem = half_out ? 2 : (word_out ? 4 : 1);
    const bool staged = !next || out_order == FLEXIQ_ORDER_NEXT_SLAB;
    const void *slab = packed_path ? static_cast<const void *>(X8) : static_cast<const void *>(X4);
    Layer::CallMaps &cm = L->call_maps;
    const bool cached = !packed && cm.slab == slab && cm.M == M && cm.Nb == Nb && cm.H == H && cm.W == W && cm.bk == p.BK &&
                        cm.im2col == (int)p.im2col + 2 * (int)patch && (!staged || (cm.staged && cm.Y == Y && cm.y_elem == y_elem));
    if (cached) {
        a_lo = a_hi = cm.a;
    } else if (!packed) {
        // one int8 slab [rows][C] (a packed-path layer at ratio 0 has it in X8_dev)
        if (patch) {
            if ((rc = make_map_nhwc(&a_hi, slab, (uint64_t)L->C, W, H, Nb, p.BK, 1u << p.pw_log2, p.patch_rows, p.BK))) return rc;
        } else if (p.im2col) {
            if ((rc = make_map_im2col(&a_hi, slab, L->C, L->C, Nb, H, W, L->R, L->S, L->stride, L->pad, p.BK, p.BK))) return rc;
        } else {
            const long long rows = L->is_conv ? (long long)Nb * H * W : M;
            if ((rc = make_map_2d(&a_hi, slab, (uint64_t)L->C, (uint64_t)rows, (uint64_t)L->C, p.BK, BM, p.BK))) return rc;
        }
        a_lo = a_hi;
    } else {
        // packed path: two values per byte, rows padded to 16 bytes, raw tiles of BK/2 bytes per row
        // (64-byte raw rows carry the 64-byte swizzle), plus the int8 slab of the 8-bit groups
        const long long pitch_lo = (long long)((C_lo / 2 + 15) / 16) * 16;
        const int lo_box = p.BK / 2, lo_swz = p.BK / 2 == 64 ? 64 : 0;
        if (p.im2col) {
            if ((rc = make_map_im2col(&a_lo, X4, C_lo / 2, pitch_lo, Nb, H, W, L->R, L->S, L->stride, L->pad, lo_box, lo_swz))) return rc;
            if (C_hi > 0 && (rc = make_map_im2col(&a_hi, X8, C_hi, C_hi, Nb, H, W, L->R, L->S, L->stride, L->pad, p.BK, p.BK))) return rc;
        } else {
            const long long rows = L->is_conv ? (long long)Nb * H * W : M;
            if ((rc = make_map_2d(&a_lo, X4, (uint64_t)C_lo / 2, (uint64_t)rows, (uint64_t)pitch_lo, lo_box, BM, lo_swz))) return rc;
            if (C_hi > 0 && (rc = make_map_2d(&a_hi, X8, (uint64_t)C_hi, (uint64_t)rows, (uint64_t)C_hi, p.BK, BM, p.BK))) return rc;
        }
        if (C_hi == 0) a_hi = a_lo;
    }
    // int8 output leaves through staged tiled bulk stores
    CUtensorMap y_map = a_hi, y_map16 = a_hi;
    p.tma_store = staged;
    if (staged && cached) {
        y_map = cm.y;
        y_map16 = cm.y16;
    } else if (staged && patch) {
        // a warp's 32 accumulator rows are bx consecutive pixels of by consecutive output rows
        const uint32_t bx = (1u << p.pw_log2) < 32u ? (1u << p.pw_log2) : 32u, by = 32u / bx;
        const uint64_t rb = (uint64_t)L->N * y_elem;
        if ((y_elem > 1 || L->N >= 32) && (rc = make_map_nhwc(&y_map, Y, rb, p.Q, p.P, Nb, 32, bx, by, 32))) return rc;
        if (y_elem > 1) y_map16 = y_map;
        else if ((rc = make_map_nhwc(&y_map16, Y, rb, p.Q, p.P, Nb, 16, bx, by, 0))) return rc;
    } else if (staged && y_elem > 1) {
        // rows of N 2- or 4-byte values addressed in bytes: a box is 32 bytes (16 or 8 columns) x 32 rows
        if ((rc = make_map_2d(&y_map, Y, (uint64_t)L->N * y_elem, (uint64_t)M, (uint64_t)L->N * y_elem, 32, 32, 32))) return rc;
        y_map16 = y_map;
    } else if (staged) {
        if (L->N >= 32 && (rc = make_map_2d(&y_map, Y, (uint64_t)L->N, (uint64_t)M, (uint64_t)L->N, 32, 32, 32))) return rc;
        if ((rc = make_map_2d(&y_map16, Y, (uint64_t)L->N, (uint64_t)M, (uint64_t)L->N, 16, 32, 0))) return rc;
    }
    if (!packed && !cached) {
        cm.slab = slab; cm.Y = staged ? Y : nullptr; cm.M = M; cm.Nb = Nb; cm.H = H; cm.W = W; cm.bk = p.BK; cm.im2col = (int)p.im2col + 2 * (int)patch;
        cm.staged = staged; cm.y_elem = y_elem; cm.a = a_hi; cm.y = y_map; cm.y16 = y_map16;
    }
    const int bi = weight_map_index(bn / cg);  // box rows = the B rows one CTA loads
    const bool conv_kind = p.im2col || p.tps > 1 || p.b_res;
    // One narrow tile per CTA and a long K: nothing overlaps across tiles, so the MMA warps share the tile
    // (SPLIT).  With several tiles per CTA the warps already work side by side on tiles of their own, and the
    // second accumulator's extra read in the epilogue would only cost (measured: +4 to +6 % on short-K shapes).
    const bool split = !packed && !patch && bn <= 128 && p.tps == 1 && p.T * (p.nb_lo + p.nb_hi) >= 8 &&
                       (long long)p.m_tiles * p.n_tiles <= sms / cg;
    if (next) record_slab(const_cast<Layer *>(next), Y, next->K_lo);   // the fused boundary writes the next layer's slab at its current ratio
    if (packed) return launch_kernel<1, 1, 1, false>(a_lo, a_hi, L->map_w4[bi], L->map_w8[bi], L->map_w8[bi], y_map, y_map16, p, sms, st);
    // multi-tap stages hold every channel in one K block: the whole weight operand is one of the three forms
    const bool one_block = p.tps > 1 || patch;   // every channel in one K block: the weight operand is one of the three forms as a whole
    const CUtensorMap &b_hi_map = one_block ? (b_whole == 0 ? L->map_w8[bi] : (b_whole == 1 ? L->map_w8m[bi] : L->map_wst[bi])) : L->map_w8[bi];
    if (one_block && b_whole == 2) p.b_tap_step = p.BK;
    if (patch) return launch_kernel<1, 0, 2, false>(a_lo, a_hi, L->map_w8m[bi], b_hi_map, L->map_wst[bi], y_map, y_map16, p, sms, st);
#define FLEXIQ_LAUNCH(CG_, KIND_, SPLIT_) launch_kernel<CG_, 0, KIND_, SPLIT_>(a_lo, a_hi, L->map_w8m[bi], b_hi_map, L->map_wst[bi], y_map, y_map16, p, sms, st)
    if (cg == 2) {
        if (conv_kind) return split ? FLEXIQ_LAUNCH(2, 1, true) : FLEXIQ_LAUNCH(2, 1, false);
        return split ? FLEXIQ_LAUNCH(2, 0, true) : FLEXIQ_LAUNCH(2, 0, false);
    }
    if (conv_kind) return split ? FLEXIQ_LAUNCH(1, 1, true) : FLEXIQ_LAUNCH(1, 1, false);
    return split ? FLEXIQ_LAUNCH(1, 0, true) : FLEXIQ_LAUNCH(1, 0, false);
#undef FLEXIQ_LAUNCH
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

extern "C" int flexiq_mixed_gemm_to_slab(flexiq_layer_t layer, const uint8_t *X4_dev, const int8_t *X8_dev,
                                         const uint8_t *x_shift_dev, int64_t M, float x_scale, flexiq_layer_t next_layer,
                                         float next_x_scale, int relu, int out_order, uint8_t *next_X4_dev, void *stream)
{
    Layer *L = as_layer(layer), *Nx = as_layer(next_layer);
    if (!L || !Nx) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (L->is_conv) return set_error(FLEXIQ_ERR_INVALID_ARG, "layer is a convolution: use flexiq_mixed_conv_to_slab");
    if (M < 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "M = %lld is negative", (long long)M);
    return run_mixed(L, X4_dev, X8_dev, x_shift_dev, M, 0, 0, 0, x_scale, next_x_scale, 0, next_X4_dev,
                     reinterpret_cast<cudaStream_t>(stream), Nx, relu, out_order);
}

extern "C" int flexiq_mixed_conv_to_slab(flexiq_layer_t layer, const uint8_t *X4_dev, const int8_t *X8_dev,
                                         const uint8_t *x_shift_dev, int Nb, int H, int W, float x_scale,
                                         flexiq_layer_t next_layer, float next_x_scale, int relu, int out_order,
                                         uint8_t *next_X4_dev, void *stream)
{
    Layer *L = as_layer(layer), *Nx = as_layer(next_layer);
    if (!L || !Nx) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (!L->is_conv) return set_error(FLEXIQ_ERR_INVALID_ARG, "layer is linear: use flexiq_mixed_gemm_to_slab");
    if (Nb < 0 || H <= 0 || W <= 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "bad activation shape Nb=%d H=%d W=%d", Nb, H, W);
    const int P = (H + 2 * L->pad - L->R) / L->stride + 1;
    const int Q = (W + 2 * L->pad - L->S) / L->stride + 1;
    if (P <= 0 || Q <= 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "filter does not fit the padded input");
    return run_mixed(L, X4_dev, X8_dev, x_shift_dev, (long long)Nb * P * Q, Nb, H, W, x_scale, next_x_scale, 0, next_X4_dev,
                     reinterpret_cast<cudaStream_t>(stream), Nx, relu, out_order);
}

extern "C" int flexiq_choose_tile(int64_t M, int N, int k_blocks, int block_k, int sm_count, int *cta_group_out, int *tile_n_out)
{
    if (M <= 0 || N <= 0 || k_blocks <= 0 || sm_count <= 0 || (block_k != 128 && block_k != 64) || !cta_group_out || !tile_n_out)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "flexiq_choose_tile: M, N, k_blocks and sm_count must be positive, block_k 128 or 64, outputs non-NULL");
    const TileChoice tc = choose_tile(M, N, k_blocks, block_k, sm_count);
    *cta_group_out = tc.cg;
    *tile_n_out = tc.bn;
    return FLEXIQ_OK;
}

extern "C" int flexiq_force_tile(int cta_group, int tile_n)
{
    if (cta_group == 0) { g_forced_tile = TileChoice{0, 0}; return FLEXIQ_OK; }
    if ((cta_group != 1 && cta_group != 2) || (tile_n != 64 && tile_n != 128 && tile_n != 192 && tile_n != 256) ||
        (cta_group == 2 && tile_n < 128))
        return set_error(FLEXIQ_ERR_INVALID_ARG, "unsupported tile: cta_group %d, tile_n %d", cta_group, tile_n);
    g_forced_tile = TileChoice{cta_group, tile_n};
    return FLEXIQ_OK;
}

extern "C" int flexiq_selftest_wait_expiry(int *result_dev, void *stream)
{
    if (!result_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "result_dev is NULL");
    int rc = check_device_sm100();
    if (rc) return rc;
    wait_expiry_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(result_dev);
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    return FLEXIQ_OK;
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

extern "C" int flexiq_layer_sync_ratio(flexiq_layer_t layer, void *stream)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    int rc = check_device_sm100();
    if (rc) return rc;
    if ((rc = check_layer_device(L))) return rc;
    return sync_straddle(L, reinterpret_cast<cudaStream_t>(stream));
}

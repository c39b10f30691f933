// Internal declarations shared by the translation units of libflexiq (host side).
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>
#include <stdarg.h>

#include "flexiq.h"

namespace flexiq {

// Box heights (rows of the B tile one CTA loads) the weight tensor maps are encoded for.
constexpr int kNumWeightMaps = 6;
constexpr int kWeightMapRows[kNumWeightMaps] = {32, 64, 96, 128, 192, 256};
inline int weight_map_index(int rows)
{
    for (int i = 0; i < kNumWeightMaps; ++i)
        if (kWeightMapRows[i] == rows) return i;
    return -1;
}

// Layer handle: everything the static part of the method produces (layout
// post-processing, weight extraction positions, cached 4-bit weights) plus the one
// run-time knob, max_4bit_ch.
struct Layer {
    uint32_t magic;
    int is_conv;
    int C;        // input-feature channels (K for a linear layer, Cin for a conv)
    int N;        // output channels
    int G;        // channel-group size
    int n_g;      // C / G
    int R, S, stride, pad;  // taps (1,1,1,0 for linear)
    int Kw;       // R*S*C: row length of the slab-order weight matrices
    int K_lo;     // max_4bit_ch, multiple of G
    int lowbit_path;
    int device;
    // device tables
    int8_t *w8;      // [N][Kw] slab-order int8 weights
    int8_t *w8m;     // [N][Kw] (w >> sw) << sw : 4-bit weights at their extraction position
    uint8_t *w4;     // [N][Kw/2] packed 4-bit weights (w >> sw)
    // Masked path: K blocks wholly below max_4bit_ch are read from w8m, K blocks wholly above it from w8.
    // Only the one block that contains the boundary (when max_4bit_ch is not a multiple of the block) needs
    // both: it lives in wst, [N][taps][BK] bytes, rewritten when the ratio changes (see straddle.cuh).
    int8_t *wst;
    int st_K_lo;                   // the max_4bit_ch wst holds as far as eager calls know; -1 = unknown
    int st_graph_seen;             // a write of wst was captured into a CUDA graph: replays rewrite wst behind
                                   // st_K_lo, so eager calls no longer trust it
    unsigned long long st_cap_id;  // capture sequence that last wrote wst, and for which max_4bit_ch
    int st_cap_K_lo;
    uint8_t *sw;     // [n_g][N] weight extraction positions
    uint8_t *sx;     // [n_g] static activation positions, slab order
    int32_t *perm;   // [n_g]
    int32_t *inv_perm;  // [n_g] slab position of each original group
    // where a producer that writes this layer's masked slab directly puts each 16-channel chunk of
    // the original channel order, and the static position of the chunk's group
    int32_t *chunk_ent;       // [C/16] by original chunk: slab position in chunks | position of the group << 24
    int32_t *chunk_ent_slab;  // [C/16] the same for a producer that already emits slab order: c | position << 24
    float *w_scale;  // [N]
    float *bias;     // [N] or nullptr
    // perm, inv_perm, chunk_ent, chunk_ent_slab and sx live in ONE device block so that a layout uploads
    // them with a single copy from the pinned mirror below
    void *tables;             // the device block
    void *tables_host;        // pinned mirror, same layout
    size_t tables_bytes;
    cudaEvent_t tables_event; // recorded after the upload: the mirror may be rewritten once it has passed
    int tables_in_flight;
    // host copies
    int32_t *perm_host;
    uint8_t *sx_host;
    // tensor maps over the weights (encoded once)
    CUtensorMap map_w8[kNumWeightMaps], map_w4[kNumWeightMaps], map_w8m[kNumWeightMaps], map_wst[kNumWeightMaps];  // one per box height
    // Per-output-channel epilogue factors.  Each table is written for one (kind of output, S_x, S_y) and
    // then only read; a table that a captured CUDA graph reads or writes is pinned to its key for good, so
    // graph replays and eager calls cannot invalidate each other's factors.  The last table is scratch:
    // used (and rewritten by every call) only when all others are pinned to other keys.
    static constexpr int kFactorTables = 4;
    struct FactorTable {
        float *alpha, *beta;
        float xs, ys;
        int mode;
        int keyed;                  // the key above is in force (always 0 for the scratch table)
        int on_device;              // an eager call has written the values
        int pinned;                 // a captured graph depends on the table keeping this key
        unsigned long long cap_id;  // capture sequence that holds a write of the values
    } factors[kFactorTables + 1];
    int factor_next;
    float *factor_mem;   // one allocation behind all tables
    int w4_pitch;    // row pitch of w4 in bytes: Kw/2 rounded up to 16
    // tensor maps of the most recent masked-path call, reused while the caller passes the same buffers
    // and shapes (encoding three maps costs more host time than the rest of a small call)
    struct CallMaps {
        const void *slab, *Y;
        long long M;
        int Nb, H, W, bk, im2col, staged, y_elem;
        CUtensorMap a, y, y16;
    } call_maps;
    // Which max_4bit_ch the caller's slab buffers were last written at (by flexiq_quantize_lower or by a
    // fused-boundary producer): a mixed_* call on a known buffer at another ratio is refused.
    struct SlabRecord { const void *ptr; int K_lo; } slab_seen[8];
    int slab_next;
    int slab_check;  // 0 = the caller opted out
};

// the slab bookkeeping above
void record_slab(Layer *L, const void *ptr, int K_lo);
int check_slab(const Layer *L, const void *ptr, const char *what);
// FLEXIQ_ERR_INVALID_ARG unless the current device is the one the handle was created on
int check_layer_device(const Layer *L);
// 0 when the stream is not being captured, else the id of the capture sequence
unsigned long long stream_capture_id(cudaStream_t st);
// masked path: does a GEMM at the layer's current max_4bit_ch read the straddle block, and must it be written first?
bool straddle_in_use(const Layer *L);
bool straddle_stale(const Layer *L, cudaStream_t st);
void straddle_written(Layer *L, cudaStream_t st);

constexpr uint32_t kLayerMagic = 0x464c5851u;  // "FLXQ"

int set_error(int code, const char *fmt, ...);
int check_device_sm100();
int device_sm_count(int device);  // cached per device
Layer *as_layer(flexiq_layer_t h);

// driver entry point for tensor-map encoding, resolved through the runtime
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                   const cuuint64_t *, const cuuint64_t *, const int *, const int *,
                                   cuuint32_t, cuuint32_t, const cuuint32_t *,
                                   CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_tiled();
EncodeIm2colFn get_encode_im2col();

// 2-D byte tensor map: rows x row_bytes (pitch_bytes between rows), box box_rows x box_bytes.
int make_map_2d(CUtensorMap *map, const void *base, uint64_t row_bytes, uint64_t rows,
                uint64_t pitch_bytes, uint32_t box_bytes, uint32_t box_rows, int swizzle_bytes);

int choose_bk(const Layer *L);
int encode_weight_maps(Layer *L);


#define FLEXIQ_CUDA_TRY(expr)                                                         \
    do {                                                                              \
        cudaError_t e__ = (expr);                                                     \
        if (e__ != cudaSuccess)                                                       \
            return ::flexiq::set_error(FLEXIQ_ERR_CUDA, "%s failed: %s", #expr,       \
                                       cudaGetErrorString(e__));                      \
    } while (0)

}  // namespace flexiq

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
    int8_t *wf;      // [N][Kw] masked path's operand: w8m for the groups below wf_K_lo, w8 for the rest
    int wf_K_lo;     // the max_4bit_ch that wf currently reflects (patched lazily, in stream order)
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
    CUtensorMap map_w8[kNumWeightMaps], map_w4[kNumWeightMaps], map_wf[kNumWeightMaps];  // one per box height
    // per-output-channel epilogue factors of the most recent call and what they were computed for
    float *alpha, *beta;
    float cache_xs, cache_ys;
    int cache_mode;
    int w4_pitch;    // row pitch of w4 in bytes: Kw/2 rounded up to 16
    // tensor maps of the most recent masked-path call, reused while the caller passes the same buffers
    // and shapes (encoding three maps costs more host time than the rest of a small call)
    struct CallMaps {
        const void *slab, *Y;
        long long M;
        int Nb, H, W, bk, im2col, staged, y_elem;
        CUtensorMap a, y, y16;
    } call_maps;
};

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

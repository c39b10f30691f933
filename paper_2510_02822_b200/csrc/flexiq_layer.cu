// Layer handles: the static part of the method.  Layout post-processing (Sec. 5),
// per-(group, output channel) weight extraction positions (Sec. 4.1, Fig. 4), cached
// 4-bit weights (Sec. 7), and the run-time ratio knob max_4bit_ch (Sec. 7).
#include "flexiq_internal.h"

#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

namespace flexiq {

static thread_local char g_err[512] = "";

int set_error(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

int check_device_sm100()
{
    static int major_of[64] = {};  // compute capability major per device ordinal, looked up once
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess)
        return set_error(FLEXIQ_ERR_CUDA, "cudaGetDevice failed: %s", cudaGetErrorString(e));
    int major = dev < 64 ? major_of[dev] : 0;
    if (major == 0) {
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess)
            return set_error(FLEXIQ_ERR_CUDA, "cudaDeviceGetAttribute failed: %s", cudaGetErrorString(e));
        if (dev < 64) major_of[dev] = major;
    }
    if (major != 10)
        return set_error(FLEXIQ_ERR_UNSUPPORTED,
                         "device compute capability %d.x is not sm_100; there is no fallback path", major);
    return FLEXIQ_OK;
}

int device_sm_count(int device)
{
    static int sms_of[64] = {};
    if (device >= 0 && device < 64 && sms_of[device]) return sms_of[device];
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (device >= 0 && device < 64) sms_of[device] = sms;
    return sms;
}

Layer *as_layer(flexiq_layer_t h)
{
    Layer *L = reinterpret_cast<Layer *>(h);
    if (L == nullptr || L->magic != kLayerMagic) return nullptr;
    return L;
}

int check_layer_device(const Layer *L)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_error(FLEXIQ_ERR_CUDA, "cudaGetDevice failed: %s", cudaGetErrorString(e));
    if (dev != L->device)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "the layer lives on device %d but device %d is current: its pointers are not valid there",
                         L->device, dev);
    return FLEXIQ_OK;
}

unsigned long long stream_capture_id(cudaStream_t st)
{
    cudaStreamCaptureStatus status = cudaStreamCaptureStatusNone;
    unsigned long long id = 0;
    if (cudaStreamGetCaptureInfo(st, &status, &id) != cudaSuccess) { cudaGetLastError(); return 0; }
    return status == cudaStreamCaptureStatusActive ? (id ? id : 1ull) : 0ull;
}

void record_slab(Layer *L, const void *ptr, int K_lo)
{
    if (!ptr) return;
    for (int i = 0; i < 8; ++i)
        if (L->slab_seen[i].ptr == ptr) { L->slab_seen[i].K_lo = K_lo; return; }
    L->slab_seen[L->slab_next] = Layer::SlabRecord{ptr, K_lo};
    L->slab_next = (L->slab_next + 1) & 7;
}

int check_slab(const Layer *L, const void *ptr, const char *what)
{
    if (!L->slab_check || !ptr) return FLEXIQ_OK;
    for (int i = 0; i < 8; ++i)
        if (L->slab_seen[i].ptr == ptr && L->slab_seen[i].K_lo != L->K_lo)
            return set_error(FLEXIQ_ERR_INVALID_ARG,
                             "%s was last written at max_4bit_ch = %d but the layer is now at %d: run flexiq_quantize_lower "
                             "again, or set the ratio the slab was written at", what, L->slab_seen[i].K_lo, L->K_lo);
    return FLEXIQ_OK;
}

// Masked path: the straddle block is read when max_4bit_ch falls inside a K block.
bool straddle_in_use(const Layer *L)
{
    return L->lowbit_path == FLEXIQ_LOWBIT_MASKED_I8 && L->K_lo < L->C && (L->K_lo % choose_bk(L)) != 0;
}
// Does wst hold the block for the current max_4bit_ch at this point of the stream?  Outside a capture the
// host's record decides, unless a captured graph may have rewritten wst since.  Inside a capture only a write
// earlier in the same capture counts, so that every graph is complete in itself and graphs of different
// ratios replay in any order.
bool straddle_stale(const Layer *L, cudaStream_t st)
{
    const unsigned long long cap = stream_capture_id(st);
    if (cap) return !(L->st_cap_id == cap && L->st_cap_K_lo == L->K_lo);
    return L->st_graph_seen || L->st_K_lo != L->K_lo;
}
void straddle_written(Layer *L, cudaStream_t st)
{
    const unsigned long long cap = stream_capture_id(st);
    if (cap) { L->st_cap_id = cap; L->st_cap_K_lo = L->K_lo; L->st_graph_seen = 1; L->st_K_lo = -1; }
    else L->st_K_lo = L->K_lo;
}

static void *driver_entry(const char *name)
{
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint(name, &fn, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
    if (qres != cudaDriverEntryPointSuccess) return nullptr;
    return fn;
}

EncodeTiledFn get_encode_tiled()
{
    static EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(driver_entry("cuTensorMapEncodeTiled"));
    return fn;
}

EncodeIm2colFn get_encode_im2col()
{
    static EncodeIm2colFn fn = reinterpret_cast<EncodeIm2colFn>(driver_entry("cuTensorMapEncodeIm2col"));
    return fn;
}

static CUtensorMapSwizzle swizzle_enum(int bytes)
{
    switch (bytes) {
        case 128: return CU_TENSOR_MAP_SWIZZLE_128B;
        case 64: return CU_TENSOR_MAP_SWIZZLE_64B;
        case 32: return CU_TENSOR_MAP_SWIZZLE_32B;
        default: return CU_TENSOR_MAP_SWIZZLE_NONE;
    }
}

int make_map_2d(CUtensorMap *map, const void *base, uint64_t row_bytes, uint64_t rows,
                uint64_t pitch_bytes, uint32_t box_bytes, uint32_t box_rows, int swizzle_bytes)
{
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return set_error(FLEXIQ_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    if ((reinterpret_cast<uintptr_t>(base) & 15) != 0 || (pitch_bytes & 15) != 0)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "tensor base %p / pitch %llu not 16-byte aligned", base,
                         (unsigned long long)pitch_bytes);
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_bytes, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box,
                     estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_enum(swizzle_bytes),
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return set_error(FLEXIQ_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d (rows %llu x %llu B, box %u x %u)",
                         (int)r, (unsigned long long)rows, (unsigned long long)row_bytes, box_rows, box_bytes);
    return FLEXIQ_OK;
}

int choose_bk(const Layer *L) { return L->C >= 128 ? 128 : 64; }

// ---------------------------------------------------------------------------------
// Weight preparation.  One thread per (slab group j, output channel n): finds the
// extraction position of the group's G weights (x all taps), then writes the three
// slab-order weight forms.  Runs once per layer.
__global__ void prep_weights_kernel(const int8_t *__restrict__ Wq, int is_conv, int C, int N, int G,
                                    int T, const int32_t *__restrict__ perm, int8_t *__restrict__ w8,
                                    int8_t *__restrict__ w8m, uint8_t *__restrict__ w4, int w4_pitch,
                                    uint8_t *__restrict__ sw)
{
    const int n_g = C / G;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)n_g * N) return;
    const int j = (int)(idx / N), n = (int)(idx % N);
    const int g = perm[j];
    const long long Kw = (long long)T * C;
    int lo = 0, hi = 0;
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < G; ++i) {
            const long long src = is_conv ? ((long long)n * T + t) * C + g * G + i
                                          : (long long)(g * G + i) * N + n;
            const int v = Wq[src];
            lo = min(lo, v);
            hi = max(hi, v);
        }
    // magnitude bits in use: bit length of hi and of ~lo; keep sign + 3 bits
    int used = 0;
    if (hi > 0) used = max(used, 32 - __clz(hi));
    if (lo < 0) used = max(used, 32 - __clz(~lo));
    const int s = used > 3 ? used - 3 : 0;
    sw[(long long)j * N + n] = (uint8_t)s;
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < G; i += 2) {
            const long long src0 = is_conv ? ((long long)n * T + t) * C + g * G + i
                                           : (long long)(g * G + i) * N + n;
            const long long src1 = is_conv ? src0 + 1 : src0 + N;
            const int v0 = Wq[src0], v1 = Wq[src1];
            const long long dst = (long long)n * Kw + (long long)t * C + j * G + i;
            w8[dst] = (int8_t)v0;
            w8[dst + 1] = (int8_t)v1;
            const int a = v0 >> s, b = v1 >> s;  // arithmetic shift: floor
            w8m[dst] = (int8_t)(a << s);
            w8m[dst + 1] = (int8_t)(b << s);
            w4[(long long)n * w4_pitch + (((long long)t * C + j * G + i) >> 1)] = (uint8_t)((a & 15) | ((b & 15) << 4));
        }
}

static int validate_perm(const int32_t *perm, int n_g)
{
    char *seen = (char *)calloc((size_t)n_g, 1);
    bool ok = true;
    for (int j = 0; j < n_g && ok; ++j) {
        if (perm[j] < 0 || perm[j] >= n_g || seen[perm[j]]) ok = false;
        else seen[perm[j]] = 1;
    }
    free(seen);
    if (!ok) return set_error(FLEXIQ_ERR_INVALID_ARG, "group_perm_host is not a permutation of 0..%d", n_g - 1);
    return FLEXIQ_OK;
}

static int validate_common(flexiq_layer_t *out, int C, int N, int G, const int8_t *Wq, const float *w_scale,
                           const int32_t *perm)
{
    if (!out) return set_error(FLEXIQ_ERR_INVALID_ARG, "out handle pointer is NULL");
    *out = nullptr;
    if (G != 16 && G != 32 && G != 64)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "group_size %d is not one of 16, 32, 64", G);
    if (C <= 0 || N <= 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "channel counts must be positive (C=%d, N=%d)", C, N);
    if (C % G != 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "input channels %d not a multiple of group_size %d", C, G);
    if (N % 16 != 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "output channels %d not a multiple of 16", N);
    if (!Wq || !w_scale || !perm) return set_error(FLEXIQ_ERR_INVALID_ARG, "Wq_dev, w_scale_dev and group_perm_host must not be NULL");
    return validate_perm(perm, C / G);
}

static void free_layer(Layer *L)
{
    if (!L) return;
    if (L->tables_in_flight) cudaEventSynchronize(L->tables_event);
    cudaFree(L->w8); cudaFree(L->w8m); cudaFree(L->w4); cudaFree(L->wst); cudaFree(L->sw);
    cudaFree(L->tables); cudaFree(L->w_scale); cudaFree(L->bias); cudaFree(L->factor_mem);
    if (L->tables_host) cudaFreeHost(L->tables_host);
    if (L->tables_event) cudaEventDestroy(L->tables_event);
    free(L->perm_host); free(L->sx_host);
    L->magic = 0;
    free(L);
}

int encode_weight_maps(Layer *L)
{
    const int bk = choose_bk(L);
    const int *bns = kWeightMapRows;
    for (int i = 0; i < kNumWeightMaps; ++i) {
        int rc = make_map_2d(&L->map_w8[i], L->w8, (uint64_t)L->Kw, (uint64_t)L->N, (uint64_t)L->Kw, bk, bns[i], bk);
        if (rc) return rc;
        rc = make_map_2d(&L->map_w8m[i], L->w8m, (uint64_t)L->Kw, (uint64_t)L->N, (uint64_t)L->Kw, bk, bns[i], bk);
        if (rc) return rc;
        const uint64_t st_row = (uint64_t)L->R * L->S * bk;   // the straddle block of every tap
        rc = make_map_2d(&L->map_wst[i], L->wst, st_row, (uint64_t)L->N, st_row, bk, bns[i], bk);
        if (rc) return rc;
        rc = make_map_2d(&L->map_w4[i], L->w4, (uint64_t)L->Kw / 2, (uint64_t)L->N, (uint64_t)L->w4_pitch, bk / 2, bns[i],
                         bk / 2 == 64 ? 64 : 0);  // raw 4-bit tiles: 64-byte rows are read row-per-thread, so they are swizzled
        if (rc) return rc;
    }
    return FLEXIQ_OK;
}

// The layout post-processing of a handle for a group order (Sec. 5): uploads the order, the
// activation positions in slab order and the chunk tables, and rebuilds the slab-order weights, their
// positions and the 4-bit cache from the original-order weights.  Stream-ordered, allocates nothing
// on the device, does not wait for the stream: the tables go up in one copy from a pinned mirror.
static int layout_layer(Layer *L, const int8_t *Wq, const int32_t *perm, const uint8_t *x_shift, cudaStream_t stream)
{
    const int n_g = L->n_g, C = L->C, G = L->G, N = L->N;
    // the pinned mirror is free again once the previous upload has read it (normally long ago)
    if (L->tables_in_flight) FLEXIQ_CUDA_TRY(cudaEventSynchronize(L->tables_event));
    memcpy(L->perm_host, perm, sizeof(int32_t) * n_g);
    for (int j = 0; j < n_g; ++j) L->sx_host[j] = x_shift ? x_shift[perm[j]] : 0;  // slab order
    const int n_c = C / 16, cpg = G / 16;
    int32_t *h_perm = static_cast<int32_t *>(L->tables_host), *h_inv = h_perm + n_g, *h_ent = h_inv + n_g, *h_ent_slab = h_ent + n_c;
    uint8_t *h_sx = reinterpret_cast<uint8_t *>(h_ent_slab + n_c);
    // chunk table: original chunk c lies in original group c*16/G, which is slab group j with perm[j] = that group
    for (int j = 0; j < n_g; ++j) {
        h_perm[j] = perm[j];
        h_inv[perm[j]] = j;
        h_sx[j] = L->sx_host[j];
        for (int i = 0; i < cpg; ++i) {
            h_ent[perm[j] * cpg + i] = (j * cpg + i) | ((int32_t)L->sx_host[j] << 24);
            h_ent_slab[j * cpg + i] = (j * cpg + i) | ((int32_t)L->sx_host[j] << 24);
        }
    }
    FLEXIQ_CUDA_TRY(cudaMemcpyAsync(L->tables, L->tables_host, L->tables_bytes, cudaMemcpyHostToDevice, stream));
    FLEXIQ_CUDA_TRY(cudaEventRecord(L->tables_event, stream));
    L->tables_in_flight = 1;
    const long long total = (long long)n_g * N;
    const int threads = 128;
    prep_weights_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, stream>>>(
        Wq, L->is_conv, C, N, G, L->R * L->S, L->perm, L->w8, L->w8m, L->w4, L->w4_pitch, L->sw);
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    L->st_K_lo = -1;   // the straddle block was cut from the previous order's weights
    L->st_cap_id = 0;
    L->slab_next = 0;  // slabs written for the previous order are no longer this layer's
    memset(L->slab_seen, 0, sizeof(L->slab_seen));
    return FLEXIQ_OK;
}

static int create_common(flexiq_layer_t *out, int is_conv, int C, int N, int R, int S, int stride, int pad,
                         int G, const int8_t *Wq, const float *w_scale, const float *bias,
                         const int32_t *perm, const uint8_t *x_shift, void *stream_)
{
    int rc = validate_common(out, C, N, G, Wq, w_scale, perm);
    if (rc) return rc;
    const int n_g = C / G;
    if (x_shift)
        for (int g = 0; g < n_g; ++g)
            if (x_shift[g] > 4) return set_error(FLEXIQ_ERR_INVALID_ARG, "x_shift_host[%d] = %d exceeds 4", g, x_shift[g]);
    if (is_conv && (R <= 0 || S <= 0 || stride <= 0 || pad < 0 || R > 15 || S > 15))
        return set_error(FLEXIQ_ERR_INVALID_ARG, "bad conv geometry R=%d S=%d stride=%d pad=%d", R, S, stride, pad);
    rc = check_device_sm100();
    if (rc) return rc;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);

    Layer *L = (Layer *)calloc(1, sizeof(Layer));
    if (!L) return set_error(FLEXIQ_ERR_CUDA, "out of host memory");
    L->magic = kLayerMagic;
    L->is_conv = is_conv; L->C = C; L->N = N; L->G = G; L->n_g = n_g;
    L->R = R; L->S = S; L->stride = stride; L->pad = pad;
    L->Kw = R * S * C; L->w4_pitch = ((L->Kw / 2 + 15) / 16) * 16; L->K_lo = 0; L->lowbit_path = FLEXIQ_LOWBIT_MASKED_I8;
    cudaGetDevice(&L->device);
    L->perm_host = (int32_t *)malloc(sizeof(int32_t) * n_g);
    L->sx_host = (uint8_t *)malloc(n_g);
    const size_t wbytes = (size_t)N * L->Kw;
#define TRY_OR_FREE(expr)                                                                        \
    do {                                                                                         \
        cudaError_t e__ = (expr);                                                                \
        if (e__ != cudaSuccess) {                                                                \
            free_layer(L);                                                                       \
            return set_error(FLEXIQ_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__));  \
        }                                                                                        \
    } while (0)
    TRY_OR_FREE(cudaMalloc(&L->w8, wbytes));
    TRY_OR_FREE(cudaMalloc(&L->w8m, wbytes));
    TRY_OR_FREE(cudaMalloc(&L->wst, (size_t)N * R * S * choose_bk(L)));
    TRY_OR_FREE(cudaMalloc(&L->w4, (size_t)N * L->w4_pitch));
    TRY_OR_FREE(cudaMemsetAsync(L->w4, 0, (size_t)N * L->w4_pitch, stream));
    TRY_OR_FREE(cudaMalloc(&L->sw, (size_t)n_g * N));
    {
        // [perm n_g | inv_perm n_g | chunk_ent n_c | chunk_ent_slab n_c] int32, then sx [n_g] bytes
        const int n_c = C / 16;
        L->tables_bytes = sizeof(int32_t) * (2 * (size_t)n_g + 2 * (size_t)n_c) + (size_t)n_g;
        TRY_OR_FREE(cudaMalloc(&L->tables, L->tables_bytes));
        TRY_OR_FREE(cudaMallocHost(&L->tables_host, L->tables_bytes));
        TRY_OR_FREE(cudaEventCreateWithFlags(&L->tables_event, cudaEventDisableTiming));
        L->perm = static_cast<int32_t *>(L->tables);
        L->inv_perm = L->perm + n_g;
        L->chunk_ent = L->inv_perm + n_g;
        L->chunk_ent_slab = L->chunk_ent + n_c;
        L->sx = reinterpret_cast<uint8_t *>(L->chunk_ent_slab + n_c);
    }
    TRY_OR_FREE(cudaMalloc(&L->w_scale, sizeof(float) * N));
    if (bias) TRY_OR_FREE(cudaMalloc(&L->bias, sizeof(float) * N));
    L->st_K_lo = -1;
    L->slab_check = 1;
    TRY_OR_FREE(cudaMalloc(&L->factor_mem, sizeof(float) * 2 * (size_t)N * (Layer::kFactorTables + 1)));
    for (int i = 0; i <= Layer::kFactorTables; ++i) {
        L->factors[i].alpha = L->factor_mem + (size_t)2 * N * i;
        L->factors[i].beta = L->factors[i].alpha + N;
    }
    TRY_OR_FREE(cudaMemcpyAsync(L->w_scale, w_scale, sizeof(float) * N, cudaMemcpyDeviceToDevice, stream));
    if (bias) TRY_OR_FREE(cudaMemcpyAsync(L->bias, bias, sizeof(float) * N, cudaMemcpyDeviceToDevice, stream));
    rc = layout_layer(L, Wq, perm, x_shift, stream);
    if (rc) { free_layer(L); return rc; }
    TRY_OR_FREE(cudaStreamSynchronize(stream));
#undef TRY_OR_FREE
    rc = encode_weight_maps(L);
    if (rc) { free_layer(L); return rc; }
    *out = reinterpret_cast<flexiq_layer_t>(L);
    return FLEXIQ_OK;
}

}  // namespace flexiq

using namespace flexiq;

extern "C" {

const char *flexiq_last_error(void) { return g_err; }

int flexiq_layer_create_linear(flexiq_layer_t *out, int K, int N, int group_size, const int8_t *Wq_dev,
                               const float *w_scale_dev, const float *bias_dev,
                               const int32_t *group_perm_host, const uint8_t *x_shift_host, void *stream)
{
    return create_common(out, 0, K, N, 1, 1, 1, 0, group_size, Wq_dev, w_scale_dev, bias_dev,
                         group_perm_host, x_shift_host, stream);
}

int flexiq_layer_create_conv(flexiq_layer_t *out, int Cin, int Cout, int R, int S, int stride, int pad,
                             int group_size, const int8_t *Wq_dev, const float *w_scale_dev,
                             const float *bias_dev, const int32_t *group_perm_host,
                             const uint8_t *x_shift_host, void *stream)
{
    return create_common(out, 1, Cin, Cout, R, S, stride, pad, group_size, Wq_dev, w_scale_dev, bias_dev,
                         group_perm_host, x_shift_host, stream);
}

int flexiq_layer_set_group_perm(flexiq_layer_t layer, const int8_t *Wq_dev, const int32_t *group_perm_host,
                                const uint8_t *x_shift_host, void *stream)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (!Wq_dev || !group_perm_host) return set_error(FLEXIQ_ERR_INVALID_ARG, "Wq_dev and group_perm_host must not be NULL");
    int rc = validate_perm(group_perm_host, L->n_g);
    if (rc) return rc;
    if (x_shift_host)
        for (int g = 0; g < L->n_g; ++g)
            if (x_shift_host[g] > 4) return set_error(FLEXIQ_ERR_INVALID_ARG, "x_shift_host[%d] = %d exceeds 4", g, x_shift_host[g]);
    rc = check_layer_device(L);
    if (rc) return rc;
    return layout_layer(L, Wq_dev, group_perm_host, x_shift_host, reinterpret_cast<cudaStream_t>(stream));
}

int flexiq_layer_destroy(flexiq_layer_t layer)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    free_layer(L);
    return FLEXIQ_OK;
}

int flexiq_layer_set_lowbit_path(flexiq_layer_t layer, int lowbit_path)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (lowbit_path != FLEXIQ_LOWBIT_MASKED_I8 && lowbit_path != FLEXIQ_LOWBIT_PACKED_U4)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "unknown lowbit_path %d", lowbit_path);
    L->lowbit_path = lowbit_path;
    return FLEXIQ_OK;
}

int flexiq_set_lowbit_ratio(flexiq_layer_t layer, float ratio)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (!(ratio >= 0.0f && ratio <= 1.0f))
        return set_error(FLEXIQ_ERR_INVALID_ARG, "ratio %f outside [0, 1]", (double)ratio);
    int n_low = (int)ceil((double)ratio * (double)L->n_g - 1e-4);
    if (n_low < 0) n_low = 0;
    if (n_low > L->n_g) n_low = L->n_g;
    L->K_lo = n_low * L->G;
    return FLEXIQ_OK;
}

int flexiq_layer_set_slab_check(flexiq_layer_t layer, int enabled)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    L->slab_check = enabled != 0;
    return FLEXIQ_OK;
}

int flexiq_get_max_4bit_ch(flexiq_layer_t layer, int *K_lo)
{
    Layer *L = as_layer(layer);
    if (!L || !K_lo) return set_error(FLEXIQ_ERR_INVALID_ARG, "bad handle or NULL output");
    *K_lo = L->K_lo;
    return FLEXIQ_OK;
}

int flexiq_x4_pitch(flexiq_layer_t layer, int K_lo, int64_t *pitch_bytes)
{
    Layer *L = as_layer(layer);
    if (!L || !pitch_bytes) return set_error(FLEXIQ_ERR_INVALID_ARG, "bad handle or NULL output");
    if (K_lo < 0 || K_lo > L->C || K_lo % L->G != 0)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "K_lo %d is not a multiple of the group size within [0, %d]", K_lo, L->C);
    *pitch_bytes = L->lowbit_path == FLEXIQ_LOWBIT_PACKED_U4 ? (int64_t)((K_lo / 2 + 15) / 16) * 16 : (int64_t)L->C;
    return FLEXIQ_OK;
}

int flexiq_layer_export(flexiq_layer_t layer, uint8_t *sw_host, int8_t *w8_host, uint8_t *w4_host)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    const size_t wbytes = (size_t)L->N * L->Kw;
    if (sw_host) FLEXIQ_CUDA_TRY(cudaMemcpy(sw_host, L->sw, (size_t)L->n_g * L->N, cudaMemcpyDeviceToHost));
    if (w8_host) FLEXIQ_CUDA_TRY(cudaMemcpy(w8_host, L->w8, wbytes, cudaMemcpyDeviceToHost));
    if (w4_host)
        FLEXIQ_CUDA_TRY(cudaMemcpy2D(w4_host, (size_t)L->Kw / 2, L->w4, (size_t)L->w4_pitch, (size_t)L->Kw / 2, (size_t)L->N,
                                     cudaMemcpyDeviceToHost));
    return FLEXIQ_OK;
}

}  // extern "C"

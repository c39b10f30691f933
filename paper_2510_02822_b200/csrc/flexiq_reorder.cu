// Residual-branch channel reorder (Sec. 5, layout post-processing step 3): a tensor that
// bypasses quantized layers on a residual connection is brought into the channel order of
// the tensor it meets, at run time, by moving whole channel groups.  A plain memory copy with
// a group permutation: one 16-byte unit per thread, gathered on the read side so that every
// store is a full, contiguous sector.
#include "flexiq_internal.h"

#include "sm100_ptx.cuh"

namespace flexiq {

// Y[m][j*G + i] = X[m][src_group[j]*G + i] for every row m, group j, channel i < G.
// units_per_group = G * elem_bytes / 16; units_per_row = C * elem_bytes / 16.
__global__ void reorder_channels_kernel(const uint4 *__restrict__ X, uint4 *__restrict__ Y, long long M, int units_per_row,
                                        int units_per_group, const int32_t *__restrict__ src_group)
{
    ptx::pdl_wait();  // X may be the previous kernel's output
    const long long total = M * units_per_row;
    const long long step = (long long)gridDim.x * blockDim.x;
    // four independent 16-byte loads in flight per thread
    for (long long base = (long long)blockIdx.x * blockDim.x + threadIdx.x; base < total; base += 4 * step) {
        uint4 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const long long idx = base + q * step;
            if (idx < total) {
                const long long m = idx / units_per_row;
                const int u = (int)(idx - m * units_per_row);
                const int j = u / units_per_group;
                const int src = __ldg(src_group + j) * units_per_group + (u - j * units_per_group);
                v[q] = __ldg(X + m * units_per_row + src);
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (base + q * step < total) Y[base + q * step] = v[q];
    }
    ptx::pdl_launch_dependents();
}

}  // namespace flexiq

using namespace flexiq;

extern "C" int flexiq_reorder_channels(flexiq_layer_t layer, const void *X_dev, int elem_bytes, int64_t M, int direction,
                                       void *Y_dev, void *stream)
{
    Layer *L = as_layer(layer);
    if (!L) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq layer handle");
    if (M < 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "M = %lld is negative", (long long)M);
    if (elem_bytes != 1 && elem_bytes != 2 && elem_bytes != 4)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "elem_bytes %d is not 1, 2 or 4", elem_bytes);
    if (direction != FLEXIQ_REORDER_TO_SLAB && direction != FLEXIQ_REORDER_FROM_SLAB)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "unknown direction %d", direction);
    if (M == 0) return FLEXIQ_OK;
    if (!X_dev || !Y_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "X_dev or Y_dev is NULL");
    if (X_dev == Y_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "the reorder cannot run in place");
    if ((reinterpret_cast<uintptr_t>(X_dev) | reinterpret_cast<uintptr_t>(Y_dev)) & 15)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "X_dev and Y_dev must be 16-byte aligned");
    int rc = check_device_sm100();
    if (rc) return rc;
    if ((rc = check_layer_device(L))) return rc;
    const int sms = device_sm_count(L->device);
    const int upr = L->C * elem_bytes / 16, upg = L->G * elem_bytes / 16;
    const long long total = (long long)M * upr;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > (long long)sms * 16) blocks = (long long)sms * 16;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks, 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.stream = reinterpret_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int32_t *src_group = direction == FLEXIQ_REORDER_TO_SLAB ? L->perm : L->inv_perm;
    FLEXIQ_CUDA_TRY(cudaLaunchKernelEx(&cfg, reorder_channels_kernel, static_cast<const uint4 *>(X_dev), static_cast<uint4 *>(Y_dev),
                                       (long long)M, upr, upg, src_group));
    return FLEXIQ_OK;
}

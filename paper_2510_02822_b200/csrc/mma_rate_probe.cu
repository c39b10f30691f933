// Stand-alone probe, not part of the library: cycles per tcgen05.mma of the 8-bit integer kind (kind::i8) and of
// the narrow floating-point kind (kind::f8f6f4, here with e4m3 and with e3m2 operand formats, fp32 accumulators),
// M = 128, K = 32 bytes per instruction, several N, issued back to back by one thread from operands resident in
// shared memory.  It answers one question of the design: does the 6-bit floating-point format, which holds the
// sixteen 4-bit values -8 .. 7 exactly, run faster than the 8-bit integer path?  Operand values do not matter for
// the timing.  Build and run:  python -m paper_2510_02822_b200.mma_rate
#include "flexiq_internal.h"
#include "sm100_ptx.cuh"
#include <stdio.h>
using namespace flexiq;

// instruction descriptor of kind::f8f6f4: fp32 accumulate, A and B of format `fmt` (0 e4m3, 1 e5m2, 3 e2m3, 4 e3m2,
// 5 e2m1), both K-major, M x N tile
__host__ __device__ constexpr uint32_t idesc_f8f6f4(int M, int N, uint32_t fmt)
{
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_f8f6f4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// kind: 0 = i8, 1 = f8f6f4 / e4m3, 2 = f8f6f4 / e3m2
__global__ void __launch_bounds__(128, 1) rate_kernel(int kind, int N, int count, long long *cycles, int *status)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *A = smem;                          // 128 rows x 128 bytes
    uint8_t *B = smem + 32768;                  // up to 256 rows x 128 bytes
    uint64_t *bar = reinterpret_cast<uint64_t *>(smem + 65536);
    uint32_t *tptr = reinterpret_cast<uint32_t *>(smem + 65536 + 64);
    const int warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < 65536 / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(smem)[i] = 0x01010101u * (i & 3);
    if (threadIdx.x == 0) { ptx::mbar_init(&bar[0], 1); ptx::fence_mbar_init(); }
    if (warp == 0) { ptx::tmem_alloc(tptr, 512); ptx::tmem_relinquish(); }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *tptr;
    if (threadIdx.x == 0) {
        const uint64_t adesc = ptx::smem_desc(ptx::smem_u32(A), 128);
        const uint64_t bdesc = ptx::smem_desc(ptx::smem_u32(B), 128);
        const uint32_t idesc = kind == 0 ? ptx::idesc_i8(128, N) : idesc_f8f6f4(128, N, kind == 1 ? 0u : 4u);
        const long long t0 = clock64();
        for (int i = 0; i < count; ++i) {
            if (kind == 0) ptx::mma_i8(tmem, adesc + 2 * (i & 3), bdesc + 2 * (i & 3), idesc, i > 0);
            else mma_f8f6f4(tmem, adesc + 2 * (i & 3), bdesc + 2 * (i & 3), idesc, i > 0);
        }
        const long long t1 = clock64();
        ptx::mma_commit(&bar[0]);
        uint32_t spins = 0;
        bool ok = true;
        while (!ptx::mbar_try_wait(&bar[0], 0)) { if (++spins > (1u << 24)) { ok = false; break; } }   // bounded
        const long long t2 = clock64();
        cycles[0] = t1 - t0;
        cycles[1] = t2 - t0;
        if (!ok) *status = 1;
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) { ptx::tc_fence_after_sync(); ptx::tmem_dealloc(tmem, 512); }
}

int main()
{
    long long *d;
    int *st;
    cudaMalloc(&d, 16);
    cudaMalloc(&st, 4);
    cudaFuncSetAttribute(rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 66560);
    const char *names[3] = {"kind::i8 (s8 x s8 -> s32)", "kind::f8f6f4 (e4m3 x e4m3 -> f32)", "kind::f8f6f4 (e3m2 x e3m2 -> f32)"};
    for (int kind = 0; kind < 3; ++kind)
        for (int N : {64, 128, 256}) {
            const int count = 512;
            cudaMemset(st, 0, 4);
            rate_kernel<<<1, 128, 66560>>>(kind, N, count, d, st);   // warm-up
            rate_kernel<<<1, 128, 66560>>>(kind, N, count, d, st);
            cudaError_t e = cudaDeviceSynchronize();
            long long h[2];
            int s = 0;
            cudaMemcpy(h, d, 16, cudaMemcpyDeviceToHost);
            cudaMemcpy(&s, st, 4, cudaMemcpyDeviceToHost);
            printf("%-36s M 128 N %3d K 32: issue %.1f cycles/MMA, complete %.1f cycles/MMA = %.0f MAC/cycle/SM (%s, status %d)\n",
                   names[kind], N, (double)h[0] / count, (double)h[1] / count, 128.0 * N * 32 * count / (double)h[1], cudaGetErrorString(e), s);
            if (e != cudaSuccess) return 1;
        }
    return 0;
}

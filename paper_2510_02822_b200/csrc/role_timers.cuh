// Role timers of the mixed GEMM kernel: development instrumentation, kept apart from the kernel source.
// The product build defines none of this (every PROF_* macro expands to nothing).  A build with
// -DFLEXIQ_PROFILE makes CTA 0 record, per warp role, the cycles it spends waiting and working, and
// exports them through flexiq_profile_counters (16 counters, meaning given where they are stored).
#pragma once

#ifdef FLEXIQ_PROFILE
#include <cuda_runtime.h>
#include "flexiq_internal.h"
namespace flexiq { __device__ long long g_prof[16]; }
#define PROF_DECL(name) long long name = 0
#define PROF_T0(t) const long long t = clock64()
#define PROF_ADD(name, t) name += clock64() - t
#define PROF_STORE(i, v) do { if (blockIdx.x == 0) ::flexiq::g_prof[i] = (v); } while (0)
extern "C" int flexiq_profile_counters(long long *out16)
{
    FLEXIQ_CUDA_TRY(cudaDeviceSynchronize());
    FLEXIQ_CUDA_TRY(cudaMemcpyFromSymbol(out16, ::flexiq::g_prof, sizeof(long long) * 16));
    return FLEXIQ_OK;
}
#else
#define PROF_DECL(name)
#define PROF_T0(t)
#define PROF_ADD(name, t)
#define PROF_STORE(i, v)
#endif

// Device helpers shared by the activation prologue and the calibration kernels: Eq. 1
// (quantization of a floating-point activation to int8) on 16 channels at a time.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "flexiq.h"

namespace flexiq {

// Eq. 1 divides by the scale.  The scale is the same for every element, so its correctly
// rounded reciprocal r = RN(1/S) is computed once per thread and each quotient follows from
// two Newton corrections with exact fused residuals:
//     t = RN(x*r);  t = RN(t + r*(x - S*t));  t = RN(t + r*(x - S*t))
// With r correctly rounded and the first corrected t faithful, the last step yields the
// correctly rounded quotient RN(x/S) (Markstein's theorem), i.e. the IEEE division result,
// at five instructions per element.  (Only the final integer matters here: results in the
// subnormal range may differ but round to 0 either way.)  Infinite inputs, or inputs whose product with
// r overflows, turn the corrections into NaN (inf - inf); the caller's clip fmaxf(NaN, lo) then yields lo,
// which is right for the negative side only.  So x is first capped at 256 S from above -- every value
// beyond it quantizes to 127 anyway -- and both infinities saturate as Eq. 1's clip says.  NaN inputs
// are excluded.
struct Divider {
    float S, r, lim;
    __device__ __forceinline__ float operator()(float x) const
    {
        x = fminf(x, lim);
        float t = __fmul_rn(x, r);
        t = __fmaf_rn(__fmaf_rn(-S, t, x), r, t);
        t = __fmaf_rn(__fmaf_rn(-S, t, x), r, t);
        return t;
    }
};
__device__ __forceinline__ Divider make_divider(float scale)
{
    Divider d;
    d.S = scale;
    d.r = __frcp_rn(scale);
    d.lim = __fmul_rn(256.0f, scale);
    return d;
}

// two int32 -> two saturated int8 in the low half, upper half taken from c's low half
__device__ __forceinline__ unsigned pack2_sat_s8(int hi, int lo, unsigned c)
{
    unsigned d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(hi), "r"(lo), "r"(c));
    return d;
}
// clip(round_half_even(t), -128, 127) of four values, packed little-endian
__device__ __forceinline__ unsigned quant4(float t0, float t1, float t2, float t3)
{
    const unsigned top = pack2_sat_s8(__float2int_rn(t3), __float2int_rn(t2), 0u);
    return pack2_sat_s8(__float2int_rn(t1), __float2int_rn(t0), top);
}

// Loads the 16 channels starting at p as fp32 (exact widening for fp16 / bf16).
template <int DTYPE>
__device__ __forceinline__ void load16(const void *p, float x[16])
{
    if (DTYPE == FLEXIQ_DTYPE_F32) {
        const float4 *v = reinterpret_cast<const float4 *>(p);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 f = __ldg(v + i);
            x[4 * i + 0] = f.x; x[4 * i + 1] = f.y; x[4 * i + 2] = f.z; x[4 * i + 3] = f.w;
        }
    } else {
        const uint4 *v = reinterpret_cast<const uint4 *>(p);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint4 u = __ldg(v + i);
            const unsigned w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (DTYPE == FLEXIQ_DTYPE_F16) {
                    const __half2 h = *reinterpret_cast<const __half2 *>(&w[k]);
                    x[8 * i + 2 * k] = __low2float(h);
                    x[8 * i + 2 * k + 1] = __high2float(h);
                } else {  // bf16: the 16 bits are the top half of an fp32
                    x[8 * i + 2 * k] = __uint_as_float(w[k] << 16);
                    x[8 * i + 2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
                }
            }
        }
    }
}

// The 16 channels of one slab chunk as four words of packed int8: q = Eq. 1 of the input,
// clipped to [lo, hi] (both integers, so clipping before the rounding gives the same value
// as clipping after it).  int8 input is only clipped.
template <int DTYPE>
__device__ __forceinline__ void quantize16(const void *p, const Divider &div, float lo, float hi, unsigned w[4])
{
    if (DTYPE == FLEXIQ_DTYPE_I8) {
        const uint4 u = __ldg(reinterpret_cast<const uint4 *>(p));
        const unsigned in[4] = {u.x, u.y, u.z, u.w};
        const int ilo = (int)lo, ihi = (int)hi;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            int b[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = max(ilo, min(ihi, (int)(signed char)((in[k] >> (8 * j)) & 0xff)));
            w[k] = pack2_sat_s8(b[1], b[0], pack2_sat_s8(b[3], b[2], 0u));
        }
    } else {
        float x[16];
        load16<DTYPE>(p, x);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float t[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) t[j] = fminf(fmaxf(div(x[4 * k + j]), lo), hi);
            w[k] = quant4(t[0], t[1], t[2], t[3]);
        }
    }
}

template <int DTYPE>
__device__ __forceinline__ size_t elem_bytes()
{
    return DTYPE == FLEXIQ_DTYPE_F32 ? 4 : (DTYPE == FLEXIQ_DTYPE_I8 ? 1 : 2);
}

}  // namespace flexiq

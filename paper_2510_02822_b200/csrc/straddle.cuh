// The masked path's straddle block (Sec. 7, run-time ratio adjustment).
//
// The masked mainloop reads whole K blocks of BK channels: a block wholly below max_4bit_ch comes from
// w8m (the 4-bit weights at their extraction positions), a block wholly above it from w8.  When
// max_4bit_ch is not a multiple of BK one block per tap holds both kinds; that block is kept in
// wst [N][taps][BK]: channels below max_4bit_ch from w8m, the rest from w8, zero beyond C.  It is the
// only weight data that depends on the ratio, at most BK bytes per output channel and tap, and it is
// written by extra blocks of the prologue launch (or by a small kernel of its own when a GEMM runs
// without one).
#pragma once
#include <stdint.h>

namespace flexiq {

struct StraddleJob {
    int8_t *wst;
    const int8_t *w8m, *w8;
    int rows;              // N * taps weight rows of C channels each
    int C, BK;
    int blk0;              // first channel of the straddle block
    int K_lo;              // max_4bit_ch
    unsigned first_block;  // prologue launches: number of straddle blocks, which come in front of the quantizing blocks
};

// one 16-byte unit of the straddle block; idx < rows * (BK / 16)
__device__ __forceinline__ void straddle_write_unit(const StraddleJob &j, long long idx)
{
    const int upb = j.BK >> 4;
    const int u = (int)(idx % upb);
    const long long row = idx / upb;
    const int c = j.blk0 + 16 * u;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (c < j.C) v = *reinterpret_cast<const uint4 *>((c < j.K_lo ? j.w8m : j.w8) + (size_t)row * j.C + c);
    *reinterpret_cast<uint4 *>(j.wst + (size_t)row * j.BK + 16 * u) = v;
}

}  // namespace flexiq

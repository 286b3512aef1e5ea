// Negative-example draws shared by the pair-list kernel and the update kernels.
#pragma once
#include "w2v_device.cuh"
#include "w2v_internal.h"

namespace w2v {

// k-th negative of the pair (centre token index i, context slot): a draw from the alias
// table, repeated while it equals the context word (Algorithms 1 and 2: "N negative word
// indices != w_O"); after kMaxRedraw collisions the next word id is taken.
__device__ __forceinline__ uint32_t draw_negative(const uint2 *__restrict__ alias, uint32_t vocab,
                                                  uint32_t k0, uint32_t k1, uint32_t i, uint32_t step_lo,
                                                  uint32_t slot, uint32_t k, uint32_t w_out,
                                                  uint32_t &draws, uint32_t &redraws)
{
    const uint32_t c2 = kPurNegative | (slot << 8);
    for (uint32_t a = 0; a < (uint32_t)kMaxRedraw; ++a) {
        const uint4 r = philox4x32_10(k0, k1, i, step_lo, c2, k | (a << 16));
        const unsigned long long r64 = ((unsigned long long)r.x << 32) | r.y;
        const uint32_t bucket = (uint32_t)__umul64hi(r64, (unsigned long long)vocab);
        const uint2 e = __ldg(alias + bucket);
        const uint32_t cand = r.z < e.x ? bucket : e.y;
        ++draws;
        if (cand != w_out) return cand;
        ++redraws;
    }
    return (w_out + 1u) % vocab;
}

// Negatives of one pair, spread over the warp: lane l holds negative l in n0 and
// negative l+32 in n1.
__device__ __forceinline__ void draw_pair_negatives(const StepParams &p, uint32_t i, uint32_t slot,
                                                    uint32_t w_out, uint32_t lane, uint32_t &n0,
                                                    uint32_t &n1, uint32_t &draws, uint32_t &redraws)
{
    n0 = 0; n1 = 0;
    if (lane < p.negatives)
        n0 = draw_negative(p.tab.alias, p.vocab, p.k0, p.k1, i, p.step_lo, slot, lane, w_out, draws, redraws);
    if (lane + 32u < p.negatives)
        n1 = draw_negative(p.tab.alias, p.vocab, p.k0, p.k1, i, p.step_lo, slot, lane + 32u, w_out, draws, redraws);
}

// Target t of a pair: t = 0 is the context word (label 1), t >= 1 negative t-1 (label 0).
__device__ __forceinline__ uint32_t pair_target(uint32_t t, uint32_t w_out, uint32_t n0, uint32_t n1,
                                                bool wide)
{
    const uint32_t src = t - 1u;
    uint32_t r = __shfl_sync(kFullMask, n0, src & 31u);
    if (wide) {
        const uint32_t r1 = __shfl_sync(kFullMask, n1, src & 31u);
        if (src >= 32u) r = r1;
    }
    return t == 0 ? w_out : r;
}

__device__ __forceinline__ void flush_draw_counts(DevState *st, uint32_t draws, uint32_t redraws)
{
    const uint32_t d = warp_sum(draws), r = warp_sum(redraws);
    if ((threadIdx.x & 31) == 0) {
        if (d) atomicAdd(&st->neg_draws, (unsigned long long)d);
        if (r) atomicAdd(&st->neg_redraws, (unsigned long long)r);
    }
}

}  // namespace w2v

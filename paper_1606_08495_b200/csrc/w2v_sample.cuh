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

// One batch of TB targets of a pair, t0..t0+TB-1: all TB row gathers are issued before the
// first dot is reduced.  `off` (in float4) is added to every row address; it is zero, see
// touch_fence.  onTarget(t, target_row, v, f) is called once per target with the gathered row
// and the full dot product.
template <int VPL, int TB, typename F>
__device__ __forceinline__ void target_batch(const StepParams &p, const Row<VPL> &u, uint32_t w_out,
                                             uint32_t n0, uint32_t n1, uint32_t lane, uint32_t t0,
                                             uint32_t off, F &&onTarget)
{
    const float4 *V4 = reinterpret_cast<const float4 *>(p.V);
    const bool wide = p.negatives > 32u;
    uint32_t tgt[TB];
    Row<VPL> v[TB];
    float f[TB];
#pragma unroll
    for (int b = 0; b < TB; ++b) {
        const uint32_t t = t0 + b;
        tgt[b] = pair_target(t, w_out, n0, n1, wide);
        if (t <= p.negatives) row_load(v[b], V4 + (size_t)tgt[b] * p.ld4 + off, p.d4, lane);
        else row_zero(v[b]);
    }
#pragma unroll
    for (int b = 0; b < TB; ++b) f[b] = row_dot_partial(u, v[b]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int b = 0; b < TB; ++b) f[b] += __shfl_xor_sync(kFullMask, f[b], o);
    }
#pragma unroll
    for (int b = 0; b < TB; ++b) {
        const uint32_t t = t0 + b;
        if (t <= p.negatives) onTarget(t, tgt[b], v[b], f[b]);
    }
}

// Walks the targets of one (centre, context) pair, t = 0..N in order, in batches of TB rows.
template <int VPL, int TB, typename F>
__device__ __forceinline__ void for_each_target(const StepParams &p, const Row<VPL> &u, uint32_t w_out,
                                                uint32_t n0, uint32_t n1, uint32_t lane, F &&onTarget)
{
    for (uint32_t t0 = 0; t0 <= p.negatives; t0 += TB)
        target_batch<VPL, TB>(p, u, w_out, n0, n1, lane, t0, 0u, onTarget);
}

// The same walk with the rows of the later batches (targets TB .. TB+kTouchAhead-1) touched
// before the first batch is gathered: they arrive in L2 while the first batch is worked on, at
// one register per row instead of the VPL*4 of a full gather, and the later batches wait for
// them through the address offset.
constexpr int kTouchAhead = 12;

template <int VPL, int TB, typename F>
__device__ __forceinline__ void for_each_target_touched(const StepParams &p, const Row<VPL> &u, uint32_t w_out,
                                                        uint32_t n0, uint32_t n1, uint32_t lane, F &&onTarget)
{
    constexpr int NCH = (VPL + 3) / 4;
    const float4 *V4 = reinterpret_cast<const float4 *>(p.V);
    const bool wide = p.negatives > 32u;
    uint32_t any = 0u;
    {
        uint32_t x[kTouchAhead][NCH];
#pragma unroll
        for (int b = 0; b < kTouchAhead; ++b) {
            const uint32_t t = (uint32_t)(TB + b);
            const uint32_t tgt = pair_target(t, w_out, n0, n1, wide);
            if (t <= p.negatives) row_touch<NCH>(x[b], V4 + (size_t)tgt * p.ld4, p.d4, lane);
            else {
#pragma unroll
                for (int k = 0; k < NCH; ++k) x[b][k] = 0u;
            }
        }
        target_batch<VPL, TB>(p, u, w_out, n0, n1, lane, 0u, 0u, onTarget);
#pragma unroll
        for (int b = 0; b < kTouchAhead; ++b) {
#pragma unroll
            for (int k = 0; k < NCH; ++k) any |= x[b][k];
        }
    }
    const uint32_t off = any & p.zero;
    for (uint32_t t0 = TB; t0 <= p.negatives; t0 += TB)
        target_batch<VPL, TB>(p, u, w_out, n0, n1, lane, t0, off, onTarget);
}

// Algorithm 2 for the output rows of one pair (or one CBOW example): v(t) += G[gi + t] * r for
// t = 0..N.  An addition that has to fetch its line costs the memory system more than one that
// finds it in L2, so the rows of a batch of targets are touched first (one word per DRAM burst,
// see row_touch) and the additions' addresses wait for the touches.  The most-hit rows collect
// in double precision (DV) instead.
constexpr int kTouchBatch = 12;

template <int VPL>
__device__ __forceinline__ void adjust_targets(const StepParams &p, const Row<VPL> &r, uint32_t w_out, uint32_t n0,
                                               uint32_t n1, unsigned long long gi, uint32_t lane)
{
    constexpr int NCH = (VPL + 3) / 4;
    float4 *V4 = reinterpret_cast<float4 *>(p.V);
    const uint32_t n1p = p.negatives + 1u;
    const bool wide = p.negatives > 32u;
    for (uint32_t t0 = 0; t0 < n1p; t0 += kTouchBatch) {
        const uint32_t nb = n1p - t0 < (uint32_t)kTouchBatch ? n1p - t0 : (uint32_t)kTouchBatch;
        const float gl = lane < nb ? __ldcg(p.G + gi + t0 + lane) : 0.f;   // lane b: coefficient of target t0 + b
        uint32_t tgt[kTouchBatch], x[kTouchBatch][NCH];
#pragma unroll
        for (int b = 0; b < kTouchBatch; ++b) {
            tgt[b] = pair_target(t0 + b, w_out, n0, n1, wide);
            if ((uint32_t)b < nb && tgt[b] >= p.hot_rows) row_touch<NCH>(x[b], V4 + (size_t)tgt[b] * p.ld4, p.d4, lane);
            else {
#pragma unroll
                for (int k = 0; k < NCH; ++k) x[b][k] = 0u;
            }
        }
#pragma unroll
        for (int b = 0; b < kTouchBatch; ++b) {
            const float g = __shfl_sync(kFullMask, gl, b);
            if ((uint32_t)b < nb) {
                if (tgt[b] < p.hot_rows) row_add_scaled_f64(p.DV + (size_t)tgt[b] * (4u * p.d4), g, r, p.d4, lane);
                else row_red_scaled(V4 + (size_t)tgt[b] * p.ld4 + touch_fence<NCH>(x[b], p.zero), g, r, p.d4, lane);
            }
        }
    }
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

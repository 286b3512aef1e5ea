// The paper's own decomposition (Section 5.1, Algorithms 1-3, Eq. (6)-(7)): every GPU holds one
// column slice of every row of U and V, all GPUs regenerate the same index sets from the seed,
// each computes the partial dot products of its slice ("dotprod"), the partials are summed over
// the GPUs, and each GPU applies the coefficients to its own columns ("adjust").
//
// A shard handle is an ordinary model whose d is the slice width, so the gather / reduce helpers
// and the snapshot passes 2 and 3 serve it unchanged.  What is new here:
//   shard_dots_kernel   Algorithm 1 on one slice; the partial dots of a pair are ADDED into the
//                       F arrays of all peers (peer pointers: the exchange of Algorithm 3,
//                       "(F+,F-) <- sum_s", is done by the kernel that produces the partials);
//   coefficients_kernel G+ = lr (1 - s(F+)), G- = -lr s(F-) from the summed dots (Algorithm 3);
//   shard_du_kernel     per-centre sums of G v(target) over the slice (Algorithm 2, input rows),
//                       reading V before pass 2 adds to it.
#include "w2v_sample.cuh"

namespace w2v {

// for_each_target of the update kernels, restated for this file: batches of TB rows in flight.
template <int VPL, int TB, typename F>
__device__ __forceinline__ void shard_for_each_target(const StepParams &p, const Row<VPL> &u, uint32_t w_out,
                                                      uint32_t n0, uint32_t n1, uint32_t lane, bool need_dot,
                                                      F &&onTarget)
{
    const float4 *V4 = reinterpret_cast<const float4 *>(p.V);
    const bool wide = p.negatives > 32u;
    for (uint32_t t0 = 0; t0 <= p.negatives; t0 += TB) {
        Row<VPL> v[TB];
        float f[TB];
#pragma unroll
        for (int b = 0; b < TB; ++b) {
            const uint32_t t = t0 + b;
            const uint32_t tgt = pair_target(t, w_out, n0, n1, wide);
            if (t <= p.negatives) row_load(v[b], V4 + (size_t)tgt * p.ld4, p.d4, lane);
            else row_zero(v[b]);
        }
        if (need_dot) {
#pragma unroll
            for (int b = 0; b < TB; ++b) f[b] = row_dot_partial(u, v[b]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                for (int b = 0; b < TB; ++b) f[b] += __shfl_xor_sync(kFullMask, f[b], o);
            }
        }
#pragma unroll
        for (int b = 0; b < TB; ++b) {
            const uint32_t t = t0 + b;
            if (t <= p.negatives) onTarget(t, v[b], need_dot ? f[b] : 0.f);
        }
    }
}

// ---- Algorithm 1 on one column slice, fused with the sum over shards -------------------------
template <int VPL, int TB>
__global__ void __launch_bounds__(kBlock)
shard_dots_kernel(StepParams p, ShardPeers peers)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const float4 *U4 = reinterpret_cast<const float4 *>(p.U);
    const uint32_t n1p = p.negatives + 1u;
    uint32_t draws = 0, redraws = 0;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, right = w >> 8;
        if (left + right == 0) continue;
        const uint32_t c = (uint32_t)p.ctok[q];
        const uint32_t i = p.cidx[q];
        Row<VPL> u;
        row_load(u, U4 + (size_t)c * p.ld4, p.d4, lane);
        unsigned long long gi = p.pair_off[q] * n1p;
        for (uint32_t pp = q - left; pp <= q + right; ++pp) {
            if (pp == q) continue;
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            uint32_t n0, n1;
            draw_pair_negatives(p, i, pp + p.window - q, w_out, lane, n0, n1, draws, redraws);
            // lane t keeps the partial dot of target t (and t + 32), so that the pair's partials
            // leave as one contiguous run of 4(1+N) bytes per peer
            float f0 = 0.f, f1 = 0.f;
            shard_for_each_target<VPL, TB>(p, u, w_out, n0, n1, lane, true,
                [&](uint32_t t, const Row<VPL> &, float f) {
                    if (lane == (t & 31u)) { if (t < 32u) f0 = f; else f1 = f; }
                });
            for (uint32_t r = 0; r < peers.n; ++r) {
                float *F = peers.F[r] + gi;
                if (lane < n1p) atomicAdd(F + lane, f0);
                if (lane + 32u < n1p) atomicAdd(F + lane + 32u, f1);
            }
            gi += n1p;
        }
    }
    flush_draw_counts(p.st, draws, redraws);
}

// ---- Algorithm 3: coefficients from the summed dot products ----------------------------------
__global__ void __launch_bounds__(256)
coefficients_kernel(const float *__restrict__ F, float *__restrict__ G, unsigned long long total,
                    uint32_t n1p, float lr)
{
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const float s = sigmoidf_exact(F[i]);
        G[i] = (i % n1p == 0) ? lr * (1.0f - s) : -lr * s;
    }
}

// ---- Algorithm 2, input rows: DU[q] = sum over the centre's targets of G v(target) -----------
// Reads V only; the additions to V happen in a later launch, so every v(target) is the
// start-of-call vector ("not updated until the end of the call").
template <int VPL, int TB>
__global__ void __launch_bounds__(kBlock)
shard_du_kernel(StepParams p)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    float4 *DU4 = reinterpret_cast<float4 *>(p.DU);
    const uint32_t n1p = p.negatives + 1u;
    uint32_t draws = 0, redraws = 0;    // regenerated draws are not counted twice
    Row<VPL> unused;
    row_zero(unused);
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, right = w >> 8;
        if (left + right == 0) continue;
        const uint32_t i = p.cidx[q];
        Row<VPL> du;
        row_zero(du);
        unsigned long long gi = p.pair_off[q] * n1p;
        for (uint32_t pp = q - left; pp <= q + right; ++pp) {
            if (pp == q) continue;
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            uint32_t n0, n1;
            draw_pair_negatives(p, i, pp + p.window - q, w_out, lane, n0, n1, draws, redraws);
            shard_for_each_target<VPL, TB>(p, unused, w_out, n0, n1, lane, false,
                [&](uint32_t t, const Row<VPL> &v, float) { row_axpy(du, __ldcg(p.G + gi + t), v); });
            gi += n1p;
        }
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const uint32_t idx = lane + 32u * v;
            if (idx < p.d4) DU4[(size_t)q * p.d4 + idx] = du.x[v];
        }
    }
}

// ==== narrow slices =============================================================================
// With 8 shards a 300-column vector leaves 36-40 columns (9-10 float4) per shard: one warp per row
// would idle two thirds of its lanes and fetch 160 bytes per request.  Here a warp is split into
// 32/GL groups of GL lanes (GL = 8 or 16, d/4 <= GL); each group works on its own target row, so
// one request gathers 2 or 4 rows.  Lane sl of a group holds float4 number sl of every row.
template <int GL>
struct Narrow {
    static constexpr int NG = 32 / GL;                      // rows side by side in a warp
    uint32_t lane, sl, grp;
    __device__ explicit Narrow(uint32_t lane_) : lane(lane_), sl(lane_ & (GL - 1)), grp(lane_ / GL) {}

    __device__ float4 load(const float4 *row, uint32_t d4, bool on) const
    {
        return (on && sl < d4) ? __ldcg(row + sl) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // sum over the lanes of a group
    __device__ static float group_sum(float x)
    {
#pragma unroll
        for (int o = GL / 2; o > 0; o >>= 1) x += __shfl_xor_sync(kFullMask, x, o);
        return x;
    }
    // sum over the groups of a warp (same sl in every group)
    __device__ static float across_groups(float x)
    {
#pragma unroll
        for (int o = GL; o < 32; o <<= 1) x += __shfl_xor_sync(kFullMask, x, o);
        return x;
    }
};

// target t of the pair for this lane (t may differ between the groups of a warp)
__device__ __forceinline__ uint32_t narrow_target(uint32_t t, uint32_t w_out, uint32_t n0, uint32_t n1,
                                                  uint32_t negatives)
{
    const uint32_t src = (t == 0 || t > negatives) ? 0u : t - 1u;
    const uint32_t a = __shfl_sync(kFullMask, n0, src & 31u);
    const uint32_t b = __shfl_sync(kFullMask, n1, src & 31u);
    return t == 0 ? w_out : (src < 32u ? a : b);
}

template <int GL, int TB>
__global__ void __launch_bounds__(kBlock)
shard_dots_narrow_kernel(StepParams p, ShardPeers peers)
{
    const Narrow<GL> nr(threadIdx.x & 31);
    constexpr int NG = Narrow<GL>::NG;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const float4 *U4 = reinterpret_cast<const float4 *>(p.U);
    const float4 *V4 = reinterpret_cast<const float4 *>(p.V);
    const uint32_t n1p = p.negatives + 1u;
    uint32_t draws = 0, redraws = 0;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, right = w >> 8;
        if (left + right == 0) continue;
        const uint32_t c = (uint32_t)p.ctok[q];
        const uint32_t i = p.cidx[q];
        const float4 u = nr.load(U4 + (size_t)c * p.ld4, p.d4, true);
        unsigned long long gi = p.pair_off[q] * n1p;
        for (uint32_t pp = q - left; pp <= q + right; ++pp) {
            if (pp == q) continue;
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            uint32_t n0, n1;
            draw_pair_negatives(p, i, pp + p.window - q, w_out, nr.lane, n0, n1, draws, redraws);
            for (uint32_t t0 = 0; t0 < n1p; t0 += TB * NG) {
                float f[TB];
                float4 v[TB];
#pragma unroll
                for (int b = 0; b < TB; ++b) {
                    const uint32_t t = t0 + b * NG + nr.grp;
                    const uint32_t tgt = narrow_target(t, w_out, n0, n1, p.negatives);
                    v[b] = nr.load(V4 + (size_t)tgt * p.ld4, p.d4, t < n1p);
                }
#pragma unroll
                for (int b = 0; b < TB; ++b)
                    f[b] = Narrow<GL>::group_sum(u.x * v[b].x + u.y * v[b].y + u.z * v[b].z + u.w * v[b].w);
#pragma unroll
                for (int b = 0; b < TB; ++b) {
                    const uint32_t t = t0 + b * NG + nr.grp;
                    if (nr.sl == 0 && t < n1p)
                        for (uint32_t r = 0; r < peers.n; ++r) atomicAdd(peers.F[r] + gi + t, f[b]);
                }
            }
            gi += n1p;
        }
    }
    flush_draw_counts(p.st, draws, redraws);
}

template <int GL, int TB>
__global__ void __launch_bounds__(kBlock)
shard_du_narrow_kernel(StepParams p)
{
    const Narrow<GL> nr(threadIdx.x & 31);
    constexpr int NG = Narrow<GL>::NG;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const float4 *V4 = reinterpret_cast<const float4 *>(p.V);
    float4 *DU4 = reinterpret_cast<float4 *>(p.DU);
    const uint32_t n1p = p.negatives + 1u;
    uint32_t draws = 0, redraws = 0;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, right = w >> 8;
        if (left + right == 0) continue;
        const uint32_t i = p.cidx[q];
        float4 du = make_float4(0.f, 0.f, 0.f, 0.f);
        unsigned long long gi = p.pair_off[q] * n1p;
        for (uint32_t pp = q - left; pp <= q + right; ++pp) {
            if (pp == q) continue;
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            uint32_t n0, n1;
            draw_pair_negatives(p, i, pp + p.window - q, w_out, nr.lane, n0, n1, draws, redraws);
            for (uint32_t t0 = 0; t0 < n1p; t0 += TB * NG) {
                float4 v[TB];
                float g[TB];
#pragma unroll
                for (int b = 0; b < TB; ++b) {
                    const uint32_t t = t0 + b * NG + nr.grp;
                    const uint32_t tgt = narrow_target(t, w_out, n0, n1, p.negatives);
                    v[b] = nr.load(V4 + (size_t)tgt * p.ld4, p.d4, t < n1p);
                    g[b] = t < n1p ? __ldcg(p.G + gi + t) : 0.f;
                }
#pragma unroll
                for (int b = 0; b < TB; ++b) {
                    du.x = fmaf(g[b], v[b].x, du.x); du.y = fmaf(g[b], v[b].y, du.y);
                    du.z = fmaf(g[b], v[b].z, du.z); du.w = fmaf(g[b], v[b].w, du.w);
                }
            }
            gi += n1p;
        }
        du.x = Narrow<GL>::across_groups(du.x); du.y = Narrow<GL>::across_groups(du.y);
        du.z = Narrow<GL>::across_groups(du.z); du.w = Narrow<GL>::across_groups(du.w);
        if (nr.grp == 0 && nr.sl < p.d4) DU4[(size_t)q * p.d4 + nr.sl] = du;
    }
}

// pass 2 of the snapshot plan for narrow slices: v(target) += G u(c), several targets per warp
template <int GL>
__global__ void __launch_bounds__(kBlock)
shard_adjust_v_narrow_kernel(StepParams p)
{
    const Narrow<GL> nr(threadIdx.x & 31);
    constexpr int NG = Narrow<GL>::NG;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const float4 *U4 = reinterpret_cast<const float4 *>(p.U);
    float4 *V4 = reinterpret_cast<float4 *>(p.V);
    const uint32_t n1p = p.negatives + 1u;
    uint32_t draws = 0, redraws = 0;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, right = w >> 8;
        if (left + right == 0) continue;
        const uint32_t c = (uint32_t)p.ctok[q];
        const uint32_t i = p.cidx[q];
        const float4 u = nr.load(U4 + (size_t)c * p.ld4, p.d4, true);
        unsigned long long gi = p.pair_off[q] * n1p;
        for (uint32_t pp = q - left; pp <= q + right; ++pp) {
            if (pp == q) continue;
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            uint32_t n0, n1;
            draw_pair_negatives(p, i, pp + p.window - q, w_out, nr.lane, n0, n1, draws, redraws);
            for (uint32_t t0 = 0; t0 < n1p; t0 += NG) {
                const uint32_t t = t0 + nr.grp;
                const uint32_t tgt = narrow_target(t, w_out, n0, n1, p.negatives);
                if (t < n1p && nr.sl < p.d4) {
                    const float g = __ldcg(p.G + gi + t);
                    if (tgt < p.hot_rows) {
                        double *a = p.DV + (size_t)tgt * (4u * p.d4) + 4u * nr.sl;
                        const double gd = (double)g;
                        atomicAdd(a + 0, gd * (double)u.x); atomicAdd(a + 1, gd * (double)u.y);
                        atomicAdd(a + 2, gd * (double)u.z); atomicAdd(a + 3, gd * (double)u.w);
                    } else {
                        red_add_f32x4(V4 + (size_t)tgt * p.ld4 + nr.sl, g * u.x, g * u.y, g * u.z, g * u.w);
                    }
                }
            }
            gi += n1p;
        }
    }
}

// ---- launchers --------------------------------------------------------------------------------
template <typename K>
static int shard_grid(K kernel, int sms)
{
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kBlock, 0) != cudaSuccess || occ < 1) occ = 1;
    return occ * sms;
}

template <int VPL>
static void shard_dots_for(const StepParams &p, const ShardPeers &peers, int sms, cudaStream_t s)
{
    constexpr int TB = VPL <= 2 ? 6 : (VPL <= 4 ? 4 : 2);
    shard_dots_kernel<VPL, TB><<<shard_grid(shard_dots_kernel<VPL, TB>, sms), kBlock, 0, s>>>(p, peers);
}

template <int VPL>
static void shard_du_for(const StepParams &p, int sms, cudaStream_t s)
{
    constexpr int TB = VPL <= 2 ? 6 : (VPL <= 4 ? 4 : 2);
    shard_du_kernel<VPL, TB><<<shard_grid(shard_du_kernel<VPL, TB>, sms), kBlock, 0, s>>>(p);
}

int launch_shard_dots(const StepParams &p, const ShardPeers &peers, int sms, cudaStream_t s)
{
    if (p.d4 <= 8) {
        shard_dots_narrow_kernel<8, 2><<<shard_grid(shard_dots_narrow_kernel<8, 2>, sms), kBlock, 0, s>>>(p, peers);
        return cudaGetLastError() != cudaSuccess ? -1 : 1;
    }
    if (p.d4 <= 16) {
        shard_dots_narrow_kernel<16, 3><<<shard_grid(shard_dots_narrow_kernel<16, 3>, sms), kBlock, 0, s>>>(p, peers);
        return cudaGetLastError() != cudaSuccess ? -1 : 1;
    }
#define CALL_DOTS(V) shard_dots_for<V>(p, peers, sms, s)
    switch ((p.d4 + 31) / 32) {
        case 1: CALL_DOTS(1); break;
        case 2: CALL_DOTS(2); break;
        case 3: CALL_DOTS(3); break;
        case 4: CALL_DOTS(4); break;
        case 5: CALL_DOTS(5); break;
        case 6: CALL_DOTS(6); break;
        case 7: CALL_DOTS(7); break;
        default: CALL_DOTS(8); break;
    }
#undef CALL_DOTS
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

int launch_shard_coefficients(const float *F, float *G, unsigned long long total, uint32_t n1p, float lr,
                              int sms, cudaStream_t s)
{
    if (total == 0) return 0;
    const unsigned long long want = (total + 255) / 256;
    const int grid = (int)(want < (unsigned long long)sms * 16 ? want : (unsigned long long)sms * 16);
    coefficients_kernel<<<grid, 256, 0, s>>>(F, G, total, n1p, lr);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

int launch_shard_du(const StepParams &p, int sms, cudaStream_t s)
{
    if (p.d4 <= 8) {
        shard_du_narrow_kernel<8, 2><<<shard_grid(shard_du_narrow_kernel<8, 2>, sms), kBlock, 0, s>>>(p);
        return cudaGetLastError() != cudaSuccess ? -1 : 1;
    }
    if (p.d4 <= 16) {
        shard_du_narrow_kernel<16, 3><<<shard_grid(shard_du_narrow_kernel<16, 3>, sms), kBlock, 0, s>>>(p);
        return cudaGetLastError() != cudaSuccess ? -1 : 1;
    }
#define CALL_DU(V) shard_du_for<V>(p, sms, s)
    switch ((p.d4 + 31) / 32) {
        case 1: CALL_DU(1); break;
        case 2: CALL_DU(2); break;
        case 3: CALL_DU(3); break;
        case 4: CALL_DU(4); break;
        case 5: CALL_DU(5); break;
        case 6: CALL_DU(6); break;
        case 7: CALL_DU(7); break;
        default: CALL_DU(8); break;
    }
#undef CALL_DU
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

int launch_shard_apply(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s)
{
    if (p.d4 > 16) return launch_snapshot_apply(p, blocks_per_sm, sms, s);
    if (p.d4 <= 8)
        shard_adjust_v_narrow_kernel<8><<<shard_grid(shard_adjust_v_narrow_kernel<8>, sms), kBlock, 0, s>>>(p);
    else
        shard_adjust_v_narrow_kernel<16><<<shard_grid(shard_adjust_v_narrow_kernel<16>, sms), kBlock, 0, s>>>(p);
    if (cudaGetLastError() != cudaSuccess) return -1;
    const int k = launch_snapshot_tail(p, blocks_per_sm, sms, s);
    return k < 0 ? -1 : 1 + k;
}

}  // namespace w2v

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
            if (peers.n == 1) {                       // a single array: nobody else adds to it, plain stores
                float *F = peers.F[0] + gi;
                if (lane < n1p) F[lane] = f0;
                if (lane + 32u < n1p) F[lane + 32u] = f1;
            } else {
                for (uint32_t r = 0; r < peers.n; ++r) {
                    float *F = peers.F[r] + gi;
                    if (lane < n1p) atomicAdd(F + lane, f0);
                    if (lane + 32u < n1p) atomicAdd(F + lane + 32u, f1);
                }
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
// start-of-call vector (Section 5.1: vectors change only when the call ends).
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
// With 8 shards a 300-column vector leaves 36-40 columns (9-10 float4) per shard.  One warp per
// row would idle two thirds of its lanes, and a pass that regenerates the negatives pair by pair
// is bound by that dependent chain (draw, alias-table read, then the rows), not by bytes.  So for
// slices of at most 16 float4 the index sets are written once per step (the pair list of
// w2v_sample_pairs: centre, context, negatives) and the passes stream over it.  A warp is split
// into 32/GL groups of GL lanes (GL = 8 or 16, d/4 <= GL); each group works on its own target row
// and lane sl of a group holds float4 number sl of every row.
template <int GL>
struct Narrow {
    static constexpr int NG = 32 / GL;                      // rows side by side in a warp
    uint32_t sl, grp;
    __device__ explicit Narrow(uint32_t lane) : sl(lane & (GL - 1)), grp(lane / GL) {}

    __device__ static float4 zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
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

// output word of target j of the list: the context for t = 0, negative t-1 otherwise
__device__ __forceinline__ uint32_t list_target(const StepParams &p, unsigned long long pair, uint32_t t)
{
    return (uint32_t)(t == 0 ? __ldg(p.l_context + pair) : __ldg(p.l_negs + pair * p.negatives + (t - 1u)));
}

// Algorithm 1 over the list: one group per target, TB targets per group in flight.
template <int GL, int TB>
__global__ void __launch_bounds__(kBlock)
shard_dots_list_kernel(StepParams p, ShardPeers peers)
{
    const Narrow<GL> nr(threadIdx.x & 31);
    const unsigned long long n1p = p.negatives + 1u;
    const unsigned long long total = p.st->pairs * n1p;
    const unsigned long long group = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) / GL;
    const unsigned long long ngroups = ((unsigned long long)gridDim.x * blockDim.x) / GL;
    const float4 *U4 = reinterpret_cast<const float4 *>(p.U);
    const float4 *V4 = reinterpret_cast<const float4 *>(p.V);
    const bool on = nr.sl < p.d4;
    // every lane of a warp runs the same number of rounds (the shuffles below are warp-wide)
    for (unsigned long long j0 = group - nr.grp; j0 < total; j0 += ngroups * TB) {
        float4 u[TB], v[TB];
        float f[TB];
#pragma unroll
        for (int b = 0; b < TB; ++b) {
            const unsigned long long j = j0 + nr.grp + (unsigned long long)b * ngroups;
            u[b] = v[b] = Narrow<GL>::zero();
            if (j < total && on) {
                const unsigned long long pair = j / n1p;
                const uint32_t t = (uint32_t)(j - pair * n1p);
                const uint32_t c = (uint32_t)__ldg(p.l_centre + pair);
                const uint32_t tgt = list_target(p, pair, t);
                u[b] = __ldg(U4 + (size_t)c * p.ld4 + nr.sl);       // U is not written during this pass
                v[b] = __ldcg(V4 + (size_t)tgt * p.ld4 + nr.sl);
            }
        }
#pragma unroll
        for (int b = 0; b < TB; ++b)
            f[b] = Narrow<GL>::group_sum(u[b].x * v[b].x + u[b].y * v[b].y + u[b].z * v[b].z + u[b].w * v[b].w);
#pragma unroll
        for (int b = 0; b < TB; ++b) {
            const unsigned long long j = j0 + nr.grp + (unsigned long long)b * ngroups;
            if (nr.sl == 0 && j < total) {
                if (peers.n == 1) peers.F[0][j] = f[b];           // a single array: plain stores
                else for (uint32_t r = 0; r < peers.n; ++r) atomicAdd(peers.F[r] + j, f[b]);
            }
        }
    }
}

// Algorithm 2, input rows: DU[q] = sum over the centre's targets of G v(target); a warp per centre,
// its groups share the centre's targets.
template <int GL, int TB>
__global__ void __launch_bounds__(kBlock)
shard_du_list_kernel(StepParams p)
{
    const Narrow<GL> nr(threadIdx.x & 31);
    constexpr int NG = Narrow<GL>::NG;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const float4 *V4 = reinterpret_cast<const float4 *>(p.V);
    float4 *DU4 = reinterpret_cast<float4 *>(p.DU);
    const uint32_t n1p = p.negatives + 1u;
    const bool on = nr.sl < p.d4;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t cnt = (w & 0xFFu) + (w >> 8);
        if (cnt == 0) continue;
        const unsigned long long pair0 = p.pair_off[q];
        const uint32_t nt = cnt * n1p;
        float4 du = Narrow<GL>::zero();
        for (uint32_t k0 = 0; k0 < nt; k0 += TB * NG) {
            float4 v[TB];
            float g[TB];
#pragma unroll
            for (int b = 0; b < TB; ++b) {
                const uint32_t k = k0 + b * NG + nr.grp;
                v[b] = Narrow<GL>::zero();
                g[b] = 0.f;
                if (k < nt && on) {
                    const uint32_t pr = k / n1p, t = k - pr * n1p;
                    const uint32_t tgt = list_target(p, pair0 + pr, t);
                    g[b] = __ldcg(p.G + pair0 * n1p + k);
                    v[b] = __ldcg(V4 + (size_t)tgt * p.ld4 + nr.sl);
                }
            }
#pragma unroll
            for (int b = 0; b < TB; ++b) {
                du.x = fmaf(g[b], v[b].x, du.x); du.y = fmaf(g[b], v[b].y, du.y);
                du.z = fmaf(g[b], v[b].z, du.z); du.w = fmaf(g[b], v[b].w, du.w);
            }
        }
        du.x = Narrow<GL>::across_groups(du.x); du.y = Narrow<GL>::across_groups(du.y);
        du.z = Narrow<GL>::across_groups(du.z); du.w = Narrow<GL>::across_groups(du.w);
        if (nr.grp == 0 && on) DU4[(size_t)q * p.d4 + nr.sl] = du;
    }
}

// Algorithm 2, output rows: v(target) += G u(c) over the list, one group per target.
template <int GL>
__global__ void __launch_bounds__(kBlock)
shard_adjust_v_list_kernel(StepParams p)
{
    const Narrow<GL> nr(threadIdx.x & 31);
    const unsigned long long n1p = p.negatives + 1u;
    const unsigned long long total = p.st->pairs * n1p;
    const unsigned long long group = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) / GL;
    const unsigned long long ngroups = ((unsigned long long)gridDim.x * blockDim.x) / GL;
    const float4 *U4 = reinterpret_cast<const float4 *>(p.U);
    float4 *V4 = reinterpret_cast<float4 *>(p.V);
    if (nr.sl >= p.d4) return;                      // no warp-wide operation below
    for (unsigned long long j = group; j < total; j += ngroups) {
        const unsigned long long pair = j / n1p;
        const uint32_t t = (uint32_t)(j - pair * n1p);
        const uint32_t c = (uint32_t)__ldg(p.l_centre + pair);
        const uint32_t tgt = list_target(p, pair, t);
        const float g = __ldcg(p.G + j);
        const float4 u = __ldg(U4 + (size_t)c * p.ld4 + nr.sl);     // U is written only by pass 3
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

// ---- barrier between the shards of a peer-to-peer exchange -----------------------------------
// Every shard keeps an array of n epoch words (one per shard) that its peers can write.  Shard
// `rank` announces epoch e by storing e into word `rank` of every shard's array, then waits until
// every word of its own array has reached e.  The stores follow a system-scope fence, so the
// additions that earlier kernels of this stream made into the peers' F arrays are visible before
// the announcement; the waits are acquire loads, so the kernels that follow see the peers'
// additions.  Epochs only grow, so nothing is ever reset, and a word already beyond e (a peer one
// step ahead) also ends the wait.  The wait has a time limit: a peer that never arrives (it
// failed on the host before its launch) makes this kernel set bit 1 of the error word and return;
// nothing traps and the context stays usable.
__global__ void __launch_bounds__(32)
peer_barrier_kernel(PeerFlags flags, uint32_t rank, uint32_t epoch, unsigned long long limit_ns, int *error)
{
    const uint32_t r = threadIdx.x;
    if (r >= flags.n) return;
    __threadfence_system();
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(flags.p[r] + rank), "r"(epoch) : "memory");
    unsigned long long t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    const uint32_t *mine = flags.p[rank] + r;
    for (uint32_t polls = 1;; ++polls) {
        uint32_t seen;
        asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(seen) : "l"(mine) : "memory");
        if ((int32_t)(seen - epoch) >= 0) break;
        if ((polls & 63u) == 0) {
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (now - t0 > limit_ns || polls > (1u << 30)) {
                atomicOr(error, 2);
                break;
            }
        }
        __nanosleep(200);
    }
}

int launch_peer_barrier(const PeerFlags &flags, uint32_t rank, uint32_t epoch, uint32_t timeout_ms, int *error,
                        cudaStream_t s)
{
    peer_barrier_kernel<<<1, 32, 0, s>>>(flags, rank, epoch, (unsigned long long)timeout_ms * 1000000ull, error);
    return cudaGetLastError() != cudaSuccess ? -1 : 1;
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
        shard_dots_list_kernel<8, 4><<<shard_grid(shard_dots_list_kernel<8, 4>, sms), kBlock, 0, s>>>(p, peers);
        return cudaGetLastError() != cudaSuccess ? -1 : 1;
    }
    if (p.d4 <= 16) {
        shard_dots_list_kernel<16, 4><<<shard_grid(shard_dots_list_kernel<16, 4>, sms), kBlock, 0, s>>>(p, peers);
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
        shard_du_list_kernel<8, 2><<<shard_grid(shard_du_list_kernel<8, 2>, sms), kBlock, 0, s>>>(p);
        return cudaGetLastError() != cudaSuccess ? -1 : 1;
    }
    if (p.d4 <= 16) {
        shard_du_list_kernel<16, 3><<<shard_grid(shard_du_list_kernel<16, 3>, sms), kBlock, 0, s>>>(p);
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
        shard_adjust_v_list_kernel<8><<<shard_grid(shard_adjust_v_list_kernel<8>, sms), kBlock, 0, s>>>(p);
    else
        shard_adjust_v_list_kernel<16><<<shard_grid(shard_adjust_v_list_kernel<16>, sms), kBlock, 0, s>>>(p);
    if (cudaGetLastError() != cudaSuccess) return -1;
    const int k = launch_snapshot_tail(p, blocks_per_sm, sms, s);
    return k < 0 ? -1 : 1 + k;
}

}  // namespace w2v

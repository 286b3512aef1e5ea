// The floating-point half of the step: gather rows, column-sliced partial dots reduced
// over the warp, sigmoid coefficients and scatter-add updates (Algorithms 1-3).
//
// One warp owns one centre token at a time.  Lane l holds float4 number l, l+32, ... of
// every row it touches -- a fixed column slice, the role a parameter-server shard has in
// the paper -- so "sum the shards' partial dot products" (Algorithm 3) is a butterfly of
// warp shuffles, and "apply the coefficients to the shard's columns" (Algorithm 2) is a
// 16-byte reduction into global memory per lane.  The centre row u(c) is read once and
// kept in registers for all its contexts and their 1+N targets.
#include "w2v_sample.cuh"

namespace w2v {

// negatives of pair number `pair` from the step's list (lane l: negative l in n0, negative l + 32 in n1)
__device__ __forceinline__ void load_pair_negatives(const StepParams &p, unsigned long long pair, uint32_t lane,
                                                    uint32_t &n0, uint32_t &n1)
{
    const int32_t *src = p.l_negs + pair * p.negatives;
    n0 = 0; n1 = 0;
    if (lane < p.negatives) n0 = (uint32_t)__ldcg(src + lane);
    if (lane + 32u < p.negatives) n1 = (uint32_t)__ldcg(src + lane + 32u);
}

// ---- Hogwild mode: one pass, updates land as they are computed ---------------------------
// LIST: the step's negatives were drawn into l_negs by a launch of their own (draw_negatives_kernel)
// and the entry of the next pair is fetched while the current pair's rows are in flight; otherwise
// every pair draws its own (small chunks, where one more launch would cost more than it saves).
template <int VPL, int TB, bool LIST>
__global__ void __launch_bounds__(kBlock)
sgns_hogwild_kernel(StepParams p)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    float4 *U4 = reinterpret_cast<float4 *>(p.U);
    float4 *V4 = reinterpret_cast<float4 *>(p.V);
    uint32_t draws = 0, redraws = 0;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, right = w >> 8;
        if (left + right == 0) continue;
        const uint32_t c = (uint32_t)p.ctok[q];
        const uint32_t i = p.cidx[q];
        Row<VPL> u, etot;
        row_load(u, U4 + (size_t)c * p.ld4, p.d4, lane);
        row_zero(etot);
        unsigned long long pair = 0, pair_end = 0;
        uint32_t nx0 = 0, nx1 = 0;
        if (LIST) {
            pair = p.pair_off[q];
            pair_end = pair + left + right;
            load_pair_negatives(p, pair, lane, nx0, nx1);
        }
        for (uint32_t pp = q - left; pp <= q + right; ++pp) {
            if (pp == q) continue;
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            uint32_t n0, n1;
            if (LIST) {
                n0 = nx0; n1 = nx1;
                if (++pair < pair_end) load_pair_negatives(p, pair, lane, nx0, nx1);
            } else {
                draw_pair_negatives(p, i, pp + p.window - q, w_out, lane, n0, n1, draws, redraws);
            }
            Row<VPL> e;
            row_zero(e);
            for_each_target<VPL, TB>(p, u, w_out, n0, n1, lane,
                [&](uint32_t t, uint32_t tgt, const Row<VPL> &v, float f) {
                    const float g = p.lr * ((t == 0 ? 1.0f : 0.0f) - sigmoidf_exact(f));
                    row_axpy(e, g, v);                                         // e += g v(t)
                    row_red_scaled(V4 + (size_t)tgt * p.ld4, g, u, p.d4, lane);  // v(t) += g u(c)
                });
            row_add(u, e);       // later pairs of this centre see the moved vector
            row_add(etot, e);
        }
        row_red_scaled(U4 + (size_t)c * p.ld4, 1.0f, etot, p.d4, lane);          // u(c) += sum e
    }
    if (!LIST) flush_draw_counts(p.st, draws, redraws);
}

// ---- snapshot mode, pass 1 (Algorithm 1 + the client's aggregation): dots and coefficients ----
// Reads only start-of-step tables.  Writes G for every target and the per-centre sum
// DU[q] = sum G v(target) (the scratch area of Algorithm 2 for the centre's own row).
// The step's negatives were drawn into l_negs by a flat launch before this one (a draw inside this
// loop puts a random read of the alias table in front of every pair's gathers); the list entry of
// the next pair is fetched while the current pair's rows are in flight.
template <int VPL, int TB>
__global__ void __launch_bounds__(kBlock)
sgns_snap_dots_kernel(StepParams p)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const float4 *U4 = reinterpret_cast<const float4 *>(p.U);
    float4 *DU4 = reinterpret_cast<float4 *>(p.DU);
    const uint32_t n1p = p.negatives + 1u;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, right = w >> 8;
        if (left + right == 0) continue;
        const uint32_t c = (uint32_t)p.ctok[q];
        Row<VPL> u, du;
        row_load(u, U4 + (size_t)c * p.ld4, p.d4, lane);
        row_zero(du);
        unsigned long long pair = p.pair_off[q], gi = pair * n1p;
        const unsigned long long pair_end = pair + left + right;
        uint32_t nx0, nx1;
        load_pair_negatives(p, pair, lane, nx0, nx1);
        for (uint32_t pp = q - left; pp <= q + right; ++pp) {
            if (pp == q) continue;
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            const uint32_t n0 = nx0, n1 = nx1;
            if (pair + 1 < pair_end) load_pair_negatives(p, pair + 1, lane, nx0, nx1);
            for_each_target_touched<VPL, TB>(p, u, w_out, n0, n1, lane,
                [&](uint32_t t, uint32_t, const Row<VPL> &v, float f) {
                    const float s = sigmoidf_exact(f);
                    const float g = t == 0 ? p.lr * (1.0f - s) : -p.lr * s;
                    if (lane == 0) p.G[gi + t] = g;
                    row_axpy(du, g, v);
                });
            gi += n1p;
            ++pair;
        }
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const uint32_t idx = lane + 32u * v;
            if (idx < p.d4) DU4[(size_t)q * p.d4 + idx] = du.x[v];
        }
    }
}

// ---- snapshot mode, pass 1 with the target rows staged in shared memory -----------------------
// The register-staged kernel above holds four rows per warp in flight (48 of its 128 registers),
// 64 per SM, and a read-only gather wants more than that.  Here the rows of a warp's targets arrive
// by `cp.async.bulk` in a ring of NG groups of RR slots in shared memory, one mbarrier per group: while
// group g is reduced from shared memory, groups g+1 .. g+NG-1 are in flight, also across the boundary
// between two centres, and no register holds a row that is still on its way.  The warp is
// its own producer: after it has consumed a group it arms the barrier and lets lanes 0..3 issue
// the copies of the group NG-1 ahead.  Two cursors walk the same sequence of (centre, group of
// targets): the issuing one ahead, the consuming one behind.  Every wait has a time limit, after
// which the warp raises status bit 1 and stops issuing and consuming (nothing is left in flight
// into shared memory that is still being waited for by anyone else: the block ends together).
constexpr int kRingMaxGroups = 8;
constexpr unsigned long long kRingWaitNs = 2000000000ull;

__device__ __forceinline__ uint32_t ring_saddr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

struct RingCursor {
    uint32_t q;            // kept position of the centre
    uint32_t left, cnt;    // contexts to the left / in all
    uint32_t k;            // next target of the centre, 0 .. cnt * (1 + N)
    unsigned long long pair0;
    bool done;
};

// moves the cursor to the next centre (at or after q) that has a context
__device__ __forceinline__ void ring_seek(const StepParams &p, RingCursor &c, uint32_t nk, uint32_t nwarps)
{
    for (; c.q < nk; c.q += nwarps) {
        const uint32_t w = p.win[c.q];
        c.left = w & 0xFFu; c.cnt = c.left + (w >> 8);
        if (c.cnt) { c.pair0 = p.pair_off[c.q]; c.k = 0; return; }
    }
    c.done = true;
}

// RR: rows per group (= per barrier); BT: threads of the one block per SM (all of its shared memory is ring)
template <int VPL, int RR, int BT>
__global__ void __launch_bounds__(BT, 1)
sgns_snap_dots_ring_kernel(StepParams p, uint32_t ngroups, uint32_t slot_bytes)
{
    constexpr int kRingRows = RR, kRingBlock = BT;
    extern __shared__ __align__(128) unsigned char ring_smem[];
    const uint32_t lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const uint32_t n1p = p.negatives + 1u;
    const uint32_t group_bytes = kRingRows * slot_bytes;
    unsigned char *slots = ring_smem + (size_t)wib * ngroups * group_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(ring_smem + (size_t)(kRingBlock / 32) * ngroups * group_bytes) + wib * kRingMaxGroups;
    const float4 *U4 = reinterpret_cast<const float4 *>(p.U);
    const float4 *V4 = reinterpret_cast<const float4 *>(p.V);
    float4 *DU4 = reinterpret_cast<float4 *>(p.DU);
    if (lane == 0)
        for (uint32_t g = 0; g < ngroups; ++g)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(ring_saddr(bars + g)), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();

    RingCursor is, co;                         // issuing and consuming cursor
    is.q = co.q = warp; is.done = co.done = false; is.k = co.k = 0; is.left = is.cnt = co.left = co.cnt = 0; is.pair0 = co.pair0 = 0;
    ring_seek(p, is, nk, nwarps);
    co = is;
    uint32_t issued = 0, consumed = 0;
    bool failed = false;

    // The next group of the issuing cursor (at most kRingRows targets of one centre) in two steps, so that
    // the loads of the target numbers are not waited for where they are issued: plan_group() reads them
    // for the group after the one that issue_group() sends off.
    uint32_t pl_rows = 0, pl_tgt = 0;
    auto plan_group = [&]() {
        pl_rows = 0;
        if (is.done) return;
        const uint32_t nt = is.cnt * n1p;
        pl_rows = nt - is.k < (uint32_t)kRingRows ? nt - is.k : (uint32_t)kRingRows;
        if (lane < pl_rows) {
            const uint32_t k = is.k + lane, pr = k / n1p, t = k - pr * n1p;
            const uint32_t pp = is.q - is.left + pr + (pr >= is.left ? 1u : 0u);
            pl_tgt = t == 0 ? (uint32_t)p.ctok[pp] : (uint32_t)__ldcg(p.l_negs + (is.pair0 + pr) * p.negatives + (t - 1u));
        }
        is.k += pl_rows;
        if (is.k >= nt) { is.q += nwarps; ring_seek(p, is, nk, nwarps); }
    };
    auto issue_group = [&]() {
        const uint32_t rows = pl_rows, tgt = pl_tgt, gi = issued % ngroups;
        // the slots were read with ordinary loads; the copies write them through the async proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (lane == 0)
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         ::"r"(ring_saddr(bars + gi)), "r"(rows * 16u * p.d4) : "memory");
        __syncwarp();
        if (lane < rows)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(ring_saddr(slots + (size_t)gi * group_bytes + (size_t)lane * slot_bytes)),
                           "l"(V4 + (size_t)tgt * p.ld4), "r"(16u * p.d4), "r"(ring_saddr(bars + gi)) : "memory");
        ++issued;
        plan_group();
    };

    plan_group();
    for (uint32_t g = 0; g + 1 < ngroups && pl_rows; ++g) issue_group();
    Row<VPL> u, du;
    row_zero(u); row_zero(du);
    while (!co.done && !failed) {
        if (pl_rows) issue_group();
        if (co.k == 0) {                       // a new centre
            row_load(u, U4 + (size_t)(uint32_t)p.ctok[co.q] * p.ld4, p.d4, lane);
            row_zero(du);
        }
        // wait for the group's rows
        const uint32_t gi = consumed % ngroups, parity = (consumed / ngroups) & 1u;
        {
            unsigned long long t0 = 0;
            for (uint32_t spin = 0;; ++spin) {
                uint32_t ok;
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok) : "r"(ring_saddr(bars + gi)), "r"(parity) : "memory");
                if (ok) break;
                if ((spin & 255u) == 255u) {
                    unsigned long long now;
                    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > kRingWaitNs) { failed = true; break; }
                }
            }
            failed = __any_sync(kFullMask, failed);
            if (failed) break;
        }
        const uint32_t nt = co.cnt * n1p;
        const uint32_t rows = nt - co.k < (uint32_t)kRingRows ? nt - co.k : (uint32_t)kRingRows;
        const float4 *slot = reinterpret_cast<const float4 *>(slots + (size_t)gi * group_bytes);
        Row<VPL> v[kRingRows];
        float f[kRingRows];
#pragma unroll
        for (int b = 0; b < kRingRows; ++b) {
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const uint32_t idx = lane + 32u * j;
                v[b].x[j] = ((uint32_t)b < rows && idx < p.d4) ? slot[(size_t)b * (slot_bytes / 16u) + idx] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            f[b] = row_dot_partial(u, v[b]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int b = 0; b < kRingRows; ++b) f[b] += __shfl_xor_sync(kFullMask, f[b], o);
        }
        const unsigned long long gbase = co.pair0 * n1p + co.k;
#pragma unroll
        for (int b = 0; b < kRingRows; ++b) {
            if ((uint32_t)b < rows) {
                const uint32_t t = (co.k + b) % n1p;
                const float sg = sigmoidf_exact(f[b]);
                const float g = t == 0 ? p.lr * (1.0f - sg) : -p.lr * sg;
                if (lane == (uint32_t)b) p.G[gbase + b] = g;
                row_axpy(du, g, v[b]);
            }
        }
        ++consumed;
        co.k += rows;
        if (co.k >= nt) {
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                const uint32_t idx = lane + 32u * j;
                if (idx < p.d4) DU4[(size_t)co.q * p.d4 + idx] = du.x[j];
            }
            co.q += nwarps;
            ring_seek(p, co, nk, nwarps);
        }
    }
    if (failed) {
        // copies already issued may still land: give them their time before the block's shared memory goes away
        for (uint32_t g = consumed; g < issued; ++g) {
            const uint32_t gi = g % ngroups, parity = (g / ngroups) & 1u;
            for (uint32_t spin = 0; spin < (1u << 20); ++spin) {
                uint32_t ok;
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok) : "r"(ring_saddr(bars + gi)), "r"(parity) : "memory");
                if (ok) break;
            }
        }
        if (lane == 0) atomicOr(&p.st->status, 2u);
    }
}

// ---- snapshot mode, pass 2 (Algorithm 2, output rows): v(target) += G u(c) ------------------
// U is still untouched, so u(c) is the start-of-step vector; V is only added to (adjust_targets).
// The negatives are read back from pass 1's list when there is one (a draw costs a random read of the
// alias table), else regenerated from the seed as the paper's adjust call does (column shards).
template <int VPL>
__global__ void __launch_bounds__(kBlock)
sgns_snap_adjust_v_kernel(StepParams p)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const float4 *U4 = reinterpret_cast<const float4 *>(p.U);
    const uint32_t n1p = p.negatives + 1u;
    uint32_t draws = 0, redraws = 0;   // regenerated draws are not counted twice
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, right = w >> 8;
        if (left + right == 0) continue;
        const uint32_t c = (uint32_t)p.ctok[q];
        const uint32_t i = p.cidx[q];
        Row<VPL> u;
        row_load(u, U4 + (size_t)c * p.ld4, p.d4, lane);
        unsigned long long pair = p.pair_off[q], gi = pair * n1p;
        for (uint32_t pp = q - left; pp <= q + right; ++pp) {
            if (pp == q) continue;
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            uint32_t n0 = 0, n1 = 0;
            if (p.keep_negs) {
                load_pair_negatives(p, pair, lane, n0, n1);
            } else {
                draw_pair_negatives(p, i, pp + p.window - q, w_out, lane, n0, n1, draws, redraws);
            }
            adjust_targets<VPL>(p, u, w_out, n0, n1, gi, lane);
            gi += n1p;
            ++pair;
        }
    }
}

// ---- snapshot mode, pass 2b: the most-hit output rows --------------------------------------
// A row that is drawn as a negative tens of thousands of times in one step would collect one
// fp32 rounding error per addition; its sum is kept in double precision instead and added
// here with a single rounding.  The sums are left at zero for the next step.
__global__ void __launch_bounds__(kBlock)
sgns_snap_apply_hot_kernel(StepParams p)
{
    const uint32_t d = 4u * p.d4, ld = 4u * p.ld4;
    const uint64_t total = (uint64_t)p.hot_rows * d;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const double x = p.DV[i];
        if (x != 0.0) {
            const uint64_t row = i / d, col = i % d;
            float *v = p.V + row * ld + col;
            *v = (float)((double)*v + x);
            p.DV[i] = 0.0;
        }
    }
}

// ---- snapshot mode, pass 3 (Algorithm 2, input rows): u(c) += DU[q] -------------------------
__global__ void __launch_bounds__(kBlock)
sgns_snap_apply_u_kernel(StepParams p)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    float4 *U4 = reinterpret_cast<float4 *>(p.U);
    const float4 *DU4 = reinterpret_cast<const float4 *>(p.DU);
    for (uint32_t q = warp; q < nk; q += nwarps) {
        if (p.win[q] == 0) continue;
        const uint32_t c = (uint32_t)p.ctok[q];
        for (uint32_t idx = lane; idx < p.d4; idx += 32) {
            const float4 x = __ldcg(DU4 + (size_t)q * p.d4 + idx);
            red_add_f32x4(U4 + (size_t)c * p.ld4 + idx, x.x, x.y, x.z, x.w);
        }
    }
}

// ---- launch shapes --------------------------------------------------------------------------
template <typename K>
static int grid_for(K kernel, uint32_t blocks_per_sm, int sms)
{
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kBlock, 0) != cudaSuccess || occ < 1)
        occ = 1;
    if (blocks_per_sm && (int)blocks_per_sm < occ) occ = (int)blocks_per_sm;
    return occ * sms;   // whole waves: a multiple of the SM count
}

// Only shapes whose gathered rows fit the register file are instantiated
// (VPL * TB float4 per lane).
constexpr int kMaxRowRegs = 16;

template <int VPL, int TB>
struct Shape {
    static void hogwild(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s)
    {
        if constexpr (VPL * TB <= kMaxRowRegs) {
            if (p.keep_negs) {
                const int grid = grid_for(sgns_hogwild_kernel<VPL, TB, true>, blocks_per_sm, sms);
                sgns_hogwild_kernel<VPL, TB, true><<<grid, kBlock, 0, s>>>(p);
            } else {
                const int grid = grid_for(sgns_hogwild_kernel<VPL, TB, false>, blocks_per_sm, sms);
                sgns_hogwild_kernel<VPL, TB, false><<<grid, kBlock, 0, s>>>(p);
            }
        }
    }
    static void snap_dots(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s)
    {
        if constexpr (VPL * TB <= kMaxRowRegs) {
            const int grid = grid_for(sgns_snap_dots_kernel<VPL, TB>, blocks_per_sm, sms);
            sgns_snap_dots_kernel<VPL, TB><<<grid, kBlock, 0, s>>>(p);
        }
    }
};

template <int VPL>
static void snap_adjust_v(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s)
{
    const int grid = grid_for(sgns_snap_adjust_v_kernel<VPL>, blocks_per_sm, sms);
    sgns_snap_adjust_v_kernel<VPL><<<grid, kBlock, 0, s>>>(p);
}

#define W2V_FOR_TB(VPL, CALL)                                        \
    switch (tb) {                                                    \
        case 1: Shape<VPL, 1>::CALL; break;                          \
        case 2: Shape<VPL, 2>::CALL; break;                          \
        case 3: Shape<VPL, 3>::CALL; break;                          \
        case 4: Shape<VPL, 4>::CALL; break;                          \
        case 6: Shape<VPL, 6>::CALL; break;                          \
        default: Shape<VPL, 8>::CALL; break;                         \
    }

#define W2V_FOR_VPL(CALL)                                            \
    switch (vpl) {                                                   \
        case 1: W2V_FOR_TB(1, CALL) break;                           \
        case 2: W2V_FOR_TB(2, CALL) break;                           \
        case 3: W2V_FOR_TB(3, CALL) break;                           \
        case 4: W2V_FOR_TB(4, CALL) break;                           \
        case 5: W2V_FOR_TB(5, CALL) break;                           \
        case 6: W2V_FOR_TB(6, CALL) break;                           \
        case 7: W2V_FOR_TB(7, CALL) break;                           \
        default: W2V_FOR_TB(8, CALL) break;                          \
    }

// rows in flight per warp: the requested value rounded down to an instantiated shape
static int pick_tb(uint32_t req, int vpl, uint32_t negatives)
{
    int tb = req ? (int)req : (vpl <= 2 ? 6 : (vpl <= 4 ? 4 : 2));
    if (tb > (int)negatives + 1) tb = (int)negatives + 1;
    if (tb > 8) tb = 8;
    while (tb > 1 && tb * vpl > kMaxRowRegs) --tb;
    if (tb == 5) tb = 4;
    if (tb == 7) tb = 6;
    return tb;
}

int launch_hogwild(const StepParams &p, uint32_t rows_in_flight, uint32_t blocks_per_sm, int sms,
                   cudaStream_t s)
{
    const int vpl = (int)((p.d4 + 31) / 32);
    const int tb = pick_tb(rows_in_flight, vpl, p.negatives);
    int launched = 1;
    if (p.keep_negs) {         // the step's negatives, drawn by a launch of their own
        const int k = launch_draw_negatives(p, const_cast<int32_t *>(p.l_negs), sms * 8, s);
        if (k < 0) return -1;
        launched += k;
    }
    W2V_FOR_VPL(hogwild(p, blocks_per_sm, sms, s))
    if (cudaGetLastError() != cudaSuccess) return -1;
    return launched;
}

int launch_snapshot_apply(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s)
{
    const int vpl = (int)((p.d4 + 31) / 32);
    switch (vpl) {
        case 1: snap_adjust_v<1>(p, blocks_per_sm, sms, s); break;
        case 2: snap_adjust_v<2>(p, blocks_per_sm, sms, s); break;
        case 3: snap_adjust_v<3>(p, blocks_per_sm, sms, s); break;
        case 4: snap_adjust_v<4>(p, blocks_per_sm, sms, s); break;
        case 5: snap_adjust_v<5>(p, blocks_per_sm, sms, s); break;
        case 6: snap_adjust_v<6>(p, blocks_per_sm, sms, s); break;
        case 7: snap_adjust_v<7>(p, blocks_per_sm, sms, s); break;
        default: snap_adjust_v<8>(p, blocks_per_sm, sms, s); break;
    }
    if (cudaGetLastError() != cudaSuccess) return -1;
    const int k = launch_snapshot_tail(p, blocks_per_sm, sms, s);
    return k < 0 ? -1 : 1 + k;
}

int launch_apply_hot(const StepParams &p, int sms, cudaStream_t s)
{
    if (!p.hot_rows) return 0;
    const uint64_t want = ((uint64_t)p.hot_rows * 4u * p.d4 + kBlock - 1) / kBlock;
    const int grid = (int)(want < (uint64_t)sms * 8 ? want : (uint64_t)sms * 8);
    sgns_snap_apply_hot_kernel<<<grid, kBlock, 0, s>>>(p);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

int launch_snapshot_tail(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s)
{
    int launched = 1;
    {
        const int k = launch_apply_hot(p, sms, s);
        if (k < 0) return -1;
        launched += k;
    }
    {
        const int grid = grid_for(sgns_snap_apply_u_kernel, blocks_per_sm, sms);
        sgns_snap_apply_u_kernel<<<grid, kBlock, 0, s>>>(p);
    }
    if (cudaGetLastError() != cudaSuccess) return -1;
    return launched;
}

// Pass 1 with the shared-memory ring, when at least three groups of rows fit a warp's share of the SM's
// shared memory (d <= 512) and the caller has not asked for a register shape; false = not launched.
template <int VPL, int RR, int BT>
static bool snap_dots_ring_for(const StepParams &p, int sms, cudaStream_t s)
{
    const uint32_t slot = 16u * p.d4;
    const size_t budget = 220u * 1024u, bars = (size_t)(BT / 32) * kRingMaxGroups * 8;
    uint32_t ng = (uint32_t)((budget - bars) / (BT / 32) / ((size_t)RR * slot));
    if (ng > (uint32_t)kRingMaxGroups) ng = kRingMaxGroups;
    if (ng < 2) return false;
    const size_t sm = (size_t)(BT / 32) * ng * RR * slot + bars;
    if (cudaFuncSetAttribute(sgns_snap_dots_ring_kernel<VPL, RR, BT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    sgns_snap_dots_ring_kernel<VPL, RR, BT><<<sms, BT, sm, s>>>(p, ng, slot);
    return true;
}

// Instantiated for rows of 260..384 columns (the paper's d = 300): 16 warps per SM, groups of four rows,
// two groups per warp (measured on the 60 M x 300 workload: 10.9 ms against 12.3 ms for the register-staged
// kernel; eight or twelve warps, or groups of two or three rows, are slower: the per-group work of the warp,
// not the bytes in flight, is then the limit).  Other widths keep the register-staged kernel.
static bool launch_snap_dots_ring(const StepParams &p, uint32_t rows_in_flight, int sms, cudaStream_t s)
{
    if (rows_in_flight) return false;                       // the caller asked for a register shape
    if ((p.d4 + 31) / 32 != 3) return false;
    return snap_dots_ring_for<3, 4, 512>(p, sms, s);
}

int launch_snapshot(const StepParams &p, uint32_t rows_in_flight, uint32_t blocks_per_sm, int sms,
                    cudaStream_t s)
{
    const int vpl = (int)((p.d4 + 31) / 32);
    const int tb = pick_tb(rows_in_flight, vpl, p.negatives);
    int launched = 1;
    if (!p.keep_negs || !p.l_negs) return -1;
    {                          // the step's negatives, drawn once for both passes
        const int k = launch_draw_negatives(p, const_cast<int32_t *>(p.l_negs), sms * 8, s);
        if (k < 0) return -1;
        launched += k;
    }
    if (!launch_snap_dots_ring(p, rows_in_flight, sms, s)) {
        W2V_FOR_VPL(snap_dots(p, blocks_per_sm, sms, s))
    }
    if (cudaGetLastError() != cudaSuccess) return -1;
    const int k = launch_snapshot_apply(p, blocks_per_sm, sms, s);
    return k < 0 ? -1 : launched + k;
}

}  // namespace w2v

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
    W2V_FOR_VPL(snap_dots(p, blocks_per_sm, sms, s))
    if (cudaGetLastError() != cudaSuccess) return -1;
    const int k = launch_snapshot_apply(p, blocks_per_sm, sms, s);
    return k < 0 ? -1 : launched + k;
}

}  // namespace w2v

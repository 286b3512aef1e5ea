// Continuous bag of words (footnote to Section 5: the paper notes that its design carries over to CBOW).
// One example per kept token q with at least one context word:
//   hbar = mean of the input vectors u(w_k) of the window's context words,
//   targets = the centre word (label 1) and N negatives != centre word (label 0),
//   f = hbar . v(t), g = lr (label - s(f)), v(t) += g hbar, every context word: u(w_k) += e / |C|
// with e = sum_t g v(t): plus lr times the exact gradient of the example's log likelihood.
// Same skeleton as the skip-gram step: a warp per centre, lane l owns float4 number l, l+32, ...
// of every row (a column slice), partial dots reduced by shuffles, updates as 16-byte reductions.
#include "w2v_sample.cuh"

namespace w2v {

// compacted position of the k-th context word of centre q (k < left: to the left of q)
__device__ __forceinline__ uint32_t context_pos(uint32_t q, uint32_t left, uint32_t k)
{
    return k < left ? q - left + k : q + 1u + (k - left);
}

// hbar = (1 / cw) * sum of the context words' input rows, TB rows in flight
template <int VPL, int TB>
__device__ __forceinline__ void context_mean(const StepParams &p, uint32_t q, uint32_t left, uint32_t cw,
                                             uint32_t lane, Row<VPL> &h, float &inv)
{
    const float4 *U4 = reinterpret_cast<const float4 *>(p.U);
    row_zero(h);
    for (uint32_t k0 = 0; k0 < cw; k0 += TB) {
        Row<VPL> r[TB];
#pragma unroll
        for (int b = 0; b < TB; ++b) {
            if (k0 + b < cw) {
                const uint32_t w = (uint32_t)p.ctok[context_pos(q, left, k0 + b)];
                row_load(r[b], U4 + (size_t)w * p.ld4, p.d4, lane);
            } else {
                row_zero(r[b]);
            }
        }
#pragma unroll
        for (int b = 0; b < TB; ++b) row_add(h, r[b]);
    }
    inv = 1.0f / (float)cw;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        h.x[v].x *= inv; h.x[v].y *= inv; h.x[v].z *= inv; h.x[v].w *= inv;
    }
}

// ---- Hogwild mode ---------------------------------------------------------------------------
template <int VPL, int TB>
__global__ void __launch_bounds__(kBlock)
cbow_hogwild_kernel(StepParams p)
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
        const uint32_t left = w & 0xFFu, cw = left + (w >> 8);
        if (cw == 0) continue;
        const uint32_t wq = (uint32_t)p.ctok[q];
        Row<VPL> h, e;
        float inv;
        context_mean<VPL, TB>(p, q, left, cw, lane, h, inv);
        uint32_t n0, n1;
        draw_pair_negatives(p, p.cidx[q], p.window, wq, lane, n0, n1, draws, redraws);   // slot of offset 0
        row_zero(e);
        for_each_target<VPL, TB>(p, h, wq, n0, n1, lane,
            [&](uint32_t t, uint32_t tgt, const Row<VPL> &v, float f) {
                const float g = p.lr * ((t == 0 ? 1.0f : 0.0f) - sigmoidf_exact(f));
                row_axpy(e, g, v);                                             // e += g v(t)
                row_red_scaled(V4 + (size_t)tgt * p.ld4, g, h, p.d4, lane);     // v(t) += g hbar
            });
        for (uint32_t k = 0; k < cw; ++k) {                                     // u(w_k) += e / |C|
            const uint32_t wk = (uint32_t)p.ctok[context_pos(q, left, k)];
            row_red_scaled(U4 + (size_t)wk * p.ld4, inv, e, p.d4, lane);
        }
    }
    flush_draw_counts(p.st, draws, redraws);
}

// ---- snapshot mode, pass 1: dots, coefficients G[q (1+N) + t], DU[q] = e / |C| -----------------
template <int VPL, int TB>
__global__ void __launch_bounds__(kBlock)
cbow_snap_dots_kernel(StepParams p)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    float4 *DU4 = reinterpret_cast<float4 *>(p.DU);
    const uint32_t n1p = p.negatives + 1u;
    uint32_t draws = 0, redraws = 0;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, cw = left + (w >> 8);
        if (cw == 0) continue;
        const uint32_t wq = (uint32_t)p.ctok[q];
        Row<VPL> h, e;
        float inv;
        context_mean<VPL, TB>(p, q, left, cw, lane, h, inv);
        uint32_t n0, n1;
        draw_pair_negatives(p, p.cidx[q], p.window, wq, lane, n0, n1, draws, redraws);
        if (p.keep_negs) {
            int32_t *dst = const_cast<int32_t *>(p.l_negs) + (size_t)q * p.negatives;     // this launch is the list's writer
            if (lane < p.negatives) dst[lane] = (int32_t)n0;
            if (lane + 32u < p.negatives) dst[lane + 32u] = (int32_t)n1;
        }
        row_zero(e);
        const size_t gi = (size_t)q * n1p;
        for_each_target_touched<VPL, TB>(p, h, wq, n0, n1, lane,
            [&](uint32_t t, uint32_t, const Row<VPL> &v, float f) {
                const float s = sigmoidf_exact(f);
                const float g = t == 0 ? p.lr * (1.0f - s) : -p.lr * s;
                if (lane == 0) p.G[gi + t] = g;
                row_axpy(e, g, v);
            });
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const uint32_t idx = lane + 32u * v;
            if (idx < p.d4)
                DU4[(size_t)q * p.d4 + idx] = make_float4(e.x[v].x * inv, e.x[v].y * inv, e.x[v].z * inv, e.x[v].w * inv);
        }
    }
    flush_draw_counts(p.st, draws, redraws);
}

// ---- snapshot mode, pass 2: v(t) += G hbar (U is still untouched, V is only added to) ---------
template <int VPL, int TB>
__global__ void __launch_bounds__(kBlock)
cbow_snap_adjust_v_kernel(StepParams p)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const uint32_t n1p = p.negatives + 1u;
    uint32_t draws = 0, redraws = 0;    // regenerated draws are not counted twice
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, cw = left + (w >> 8);
        if (cw == 0) continue;
        const uint32_t wq = (uint32_t)p.ctok[q];
        Row<VPL> h;
        float inv;
        context_mean<VPL, TB>(p, q, left, cw, lane, h, inv);
        uint32_t n0 = 0, n1 = 0;
        if (p.keep_negs) {
            const int32_t *src = p.l_negs + (size_t)q * p.negatives;
            if (lane < p.negatives) n0 = (uint32_t)__ldcg(src + lane);
            if (lane + 32u < p.negatives) n1 = (uint32_t)__ldcg(src + lane + 32u);
        } else {
            draw_pair_negatives(p, p.cidx[q], p.window, wq, lane, n0, n1, draws, redraws);
        }
        adjust_targets<VPL>(p, h, wq, n0, n1, (unsigned long long)q * n1p, lane);
    }
}

// ---- snapshot mode, pass 3: every context word of q gets DU[q] ---------------------------------
__global__ void __launch_bounds__(kBlock)
cbow_snap_apply_ctx_kernel(StepParams p)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    float4 *U4 = reinterpret_cast<float4 *>(p.U);
    const float4 *DU4 = reinterpret_cast<const float4 *>(p.DU);
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, cw = left + (w >> 8);
        if (cw == 0) continue;
        for (uint32_t idx = lane; idx < p.d4; idx += 32) {
            const float4 x = __ldcg(DU4 + (size_t)q * p.d4 + idx);
            for (uint32_t k = 0; k < cw; ++k) {
                const uint32_t wk = (uint32_t)p.ctok[context_pos(q, left, k)];
                red_add_f32x4(U4 + (size_t)wk * p.ld4 + idx, x.x, x.y, x.z, x.w);
            }
        }
    }
}

// ---- the examples as lists (centre word and negatives; the contexts are those of the pair list) ----
__global__ void __launch_bounds__(kBlock)
cbow_emit_kernel(StepParams p, int32_t *__restrict__ centre, int32_t *__restrict__ negs, uint64_t cap)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    uint32_t draws = 0, redraws = 0;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        if (p.win[q] == 0) continue;
        const uint32_t wq = (uint32_t)p.ctok[q];
        uint32_t n0, n1;
        draw_pair_negatives(p, p.cidx[q], p.window, wq, lane, n0, n1, draws, redraws);
        const unsigned long long ex = p.pair_off[q];           // example number (scan of "has a context")
        if (ex < cap) {
            if (lane == 0) centre[ex] = (int32_t)wq;
            if (lane < p.negatives) negs[ex * p.negatives + lane] = (int32_t)n0;
            if (lane + 32u < p.negatives) negs[ex * p.negatives + lane + 32u] = (int32_t)n1;
        }
    }
    flush_draw_counts(p.st, draws, redraws);
}

// ---- launchers --------------------------------------------------------------------------------
template <typename K>
static int cbow_grid(K kernel, uint32_t blocks_per_sm, int sms)
{
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kBlock, 0) != cudaSuccess || occ < 1) occ = 1;
    if (blocks_per_sm && (int)blocks_per_sm < occ) occ = (int)blocks_per_sm;
    return occ * sms;
}

template <int VPL>
struct CbowShape {
    static constexpr int TB = VPL <= 2 ? 6 : (VPL <= 4 ? 4 : 2);
    static void hogwild(const StepParams &p, uint32_t bps, int sms, cudaStream_t s)
    {
        cbow_hogwild_kernel<VPL, TB><<<cbow_grid(cbow_hogwild_kernel<VPL, TB>, bps, sms), kBlock, 0, s>>>(p);
    }
    static void snapshot(const StepParams &p, uint32_t bps, int sms, cudaStream_t s)
    {
        cbow_snap_dots_kernel<VPL, TB><<<cbow_grid(cbow_snap_dots_kernel<VPL, TB>, bps, sms), kBlock, 0, s>>>(p);
        cbow_snap_adjust_v_kernel<VPL, TB><<<cbow_grid(cbow_snap_adjust_v_kernel<VPL, TB>, bps, sms), kBlock, 0, s>>>(p);
    }
};

#define W2V_CBOW_VPL(CALL)                               \
    switch ((p.d4 + 31) / 32) {                          \
        case 1: CbowShape<1>::CALL; break;               \
        case 2: CbowShape<2>::CALL; break;               \
        case 3: CbowShape<3>::CALL; break;               \
        case 4: CbowShape<4>::CALL; break;               \
        case 5: CbowShape<5>::CALL; break;               \
        case 6: CbowShape<6>::CALL; break;               \
        case 7: CbowShape<7>::CALL; break;               \
        default: CbowShape<8>::CALL; break;              \
    }

int launch_cbow_hogwild(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s)
{
    W2V_CBOW_VPL(hogwild(p, blocks_per_sm, sms, s))
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

int launch_cbow_snapshot(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s)
{
    W2V_CBOW_VPL(snapshot(p, blocks_per_sm, sms, s))
    if (cudaGetLastError() != cudaSuccess) return -1;
    const int k = launch_apply_hot(p, sms, s);
    if (k < 0) return -1;
    cbow_snap_apply_ctx_kernel<<<cbow_grid(cbow_snap_apply_ctx_kernel, blocks_per_sm, sms), kBlock, 0, s>>>(p);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 3 + k;
}

int launch_cbow_emit(const StepParams &p, int32_t *centre, int32_t *negs, uint64_t cap, int grid, cudaStream_t s)
{
    cbow_emit_kernel<<<grid, kBlock, 0, s>>>(p, centre, negs, cap);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

}  // namespace w2v

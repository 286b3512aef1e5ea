// Retrieval by cosine similarity over the trained vectors (Section 2: "calculating cosine
// similarity between the ad vector and all query vectors.  The K queries with the highest
// similarity are retrieved"; Section 7.2: K = 30 nearest, kept only above tau = 0.65).
//
// For a block of BQ query rows the kernel streams the candidate rows in tiles of BC, forms the
// BQ x BC dot products in registers (a 16 x 16 thread grid, each thread a (BQ/16) x 8 patch; both
// operands staged through shared memory, k-major), scales them by the inverse norms and feeds the
// ones that can still enter a query's list into that query's sorted top-K list in shared memory.
// All arithmetic is fp32 on the CUDA cores: cosines agree with a double-precision evaluation to
// ~1e-6, which the threshold and the ranking need; the tensor cores' TF32 inputs would not give that.
#include "w2v_device.cuh"
#include "w2v_internal.h"

namespace w2v {

constexpr int kTopkBC = 128;          // candidate rows per tile
constexpr int kTopkKC = 16;           // columns per shared-memory chunk
constexpr int kTopkPad = 4;           // keeps 16-byte alignment of the k-major rows
constexpr int kTopkThreads = 256;
constexpr int kTopkPush = 16;         // at most 16 threads offer a candidate to one query per round

// 1 / |x| per candidate row (0 for a zero row): one warp per row.
__global__ void __launch_bounds__(kBlock)
row_inv_norm_kernel(const float *__restrict__ table, uint32_t d4, uint32_t ld4, uint64_t lo, uint64_t count,
                    float *__restrict__ inv_norm)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const float4 *T4 = reinterpret_cast<const float4 *>(table);
    for (uint64_t a = warp; a < count; a += nwarps) {
        const float4 *row = T4 + (lo + a) * ld4;
        float s = 0.f;
        for (uint32_t j = lane; j < d4; j += 32) {
            const float4 x = __ldcg(row + j);
            s = fmaf(x.x, x.x, s); s = fmaf(x.y, x.y, s); s = fmaf(x.z, x.z, s); s = fmaf(x.w, x.w, s);
        }
        s = warp_sum(s);
        if (lane == 0) inv_norm[a] = s > 0.f ? 1.0f / sqrtf(s) : 0.f;
    }
}

// Does (score a, id ia) rank ahead of (score b, id ib)?  Larger cosine first, then smaller id.
__device__ __forceinline__ bool ranks_ahead(float a, long long ia, float b, long long ib)
{
    return a > b || (a == b && ia < ib);
}

// Warp-wide insertion of one item into a query's sorted list (K <= 64: lane l owns slots l, l+32).
__device__ __forceinline__ void list_insert(float *sc, long long *id, uint32_t &have, uint32_t K, float c,
                                            long long cid, uint32_t lane)
{
    // position = number of entries that rank ahead of the item
    uint32_t ahead = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t s = lane + 32u * h;
        const bool a = s < have && ranks_ahead(sc[s], id[s], c, cid);
        ahead += __popc(__ballot_sync(kFullMask, a));
    }
    if (ahead >= K) return;
    const uint32_t last = have < K ? have : K - 1u;        // slot that receives the shifted tail
    float ns[2]; long long ni[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t s = lane + 32u * h;
        if (s > ahead && s <= last) { ns[h] = sc[s - 1]; ni[h] = id[s - 1]; }
    }
    __syncwarp();
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t s = lane + 32u * h;
        if (s > ahead && s <= last) { sc[s] = ns[h]; id[s] = ni[h]; }
        else if (s == ahead) { sc[s] = c; id[s] = cid; }
    }
    __syncwarp();
    if (have < K) ++have;
}

struct TopkParams {
    const float *table;
    const long long *queries;     // [m] row numbers; outside [0, vocab) gives an empty result
    const float *inv_norm;        // [cand_hi - cand_lo]
    float *part_cos;              // [splits][m][K] partial lists (sorted), or the final output
    long long *part_ids;
    uint64_t m, vocab, cand_lo, cand_hi;
    uint32_t d4, ld4, K, splits;
    float tau;
};

template <int BQ>
__global__ void __launch_bounds__(kTopkThreads)
topk_cosine_kernel(TopkParams p)
{
    constexpr int TQ = BQ / 16;                              // query rows per thread
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t d = 4u * p.d4;
    // layout: Qs[d][BQ] | Cs[KC][BC+pad] | list_sc[BQ][K] | list_id[BQ][K] | push_c[BQ][16] | push_i[BQ][16]
    //         | qinv[BQ] | thr[BQ] | have[BQ] | npush[BQ] | qrow[BQ]
    float *Qs = reinterpret_cast<float *>(smem_raw);
    float *Cs = Qs + (size_t)d * BQ;
    long long *list_id = reinterpret_cast<long long *>(Cs + kTopkKC * (kTopkBC + kTopkPad));
    long long *push_i = list_id + (size_t)BQ * p.K;
    long long *qrow = push_i + BQ * kTopkPush;
    float *list_sc = reinterpret_cast<float *>(qrow + BQ);
    float *push_c = list_sc + (size_t)BQ * p.K;
    float *qinv = push_c + BQ * kTopkPush;
    float *thr = qinv + BQ;
    uint32_t *have = reinterpret_cast<uint32_t *>(thr + BQ);
    uint32_t *npush = have + BQ;

    const uint32_t tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint32_t tx = tid & 15, ty = tid >> 4;
    const uint64_t q0 = (uint64_t)blockIdx.x * BQ;
    // this block's share of the candidates: whole tiles
    const uint64_t nc = p.cand_hi - p.cand_lo;
    const uint64_t tiles = (nc + kTopkBC - 1) / kTopkBC;
    const uint64_t t_lo = tiles * blockIdx.y / p.splits, t_hi = tiles * (blockIdx.y + 1) / p.splits;

    // ---- query block: rows into Qs (k-major), norms, empty lists ----
    for (uint32_t i = tid; i < (uint32_t)BQ; i += kTopkThreads) {
        long long r = q0 + i < p.m ? p.queries[q0 + i] : -1;
        if (r < 0 || (unsigned long long)r >= p.vocab) r = -1;
        qrow[i] = r; have[i] = 0; npush[i] = 0; thr[i] = p.tau;
    }
    __syncthreads();
    for (uint32_t e = tid; e < (uint32_t)BQ * p.d4; e += kTopkThreads) {
        const uint32_t i = e / p.d4, j4 = e % p.d4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (qrow[i] >= 0) x = __ldcg(reinterpret_cast<const float4 *>(p.table) + (size_t)qrow[i] * p.ld4 + j4);
        Qs[(4 * j4 + 0) * BQ + i] = x.x; Qs[(4 * j4 + 1) * BQ + i] = x.y;
        Qs[(4 * j4 + 2) * BQ + i] = x.z; Qs[(4 * j4 + 3) * BQ + i] = x.w;
    }
    __syncthreads();
    for (uint32_t i = wid; i < (uint32_t)BQ; i += kTopkThreads / 32) {
        float s = 0.f;
        for (uint32_t k = lane; k < d; k += 32) s = fmaf(Qs[k * BQ + i], Qs[k * BQ + i], s);
        s = warp_sum(s);
        if (lane == 0) qinv[i] = s > 0.f ? 1.0f / sqrtf(s) : 0.f;
    }
    __syncthreads();

    for (uint64_t tile = t_lo; tile < t_hi; ++tile) {
        const uint64_t c0 = tile * kTopkBC;                  // first candidate of the tile (relative)
        float acc[TQ][8];
#pragma unroll
        for (int a = 0; a < TQ; ++a)
#pragma unroll
            for (int b = 0; b < 8; ++b) acc[a][b] = 0.f;
        for (uint32_t k0 = 0; k0 < d; k0 += kTopkKC) {
            // stage candidate columns k0 .. k0+KC of the tile, transposed
            __syncthreads();
#pragma unroll
            for (int rep = 0; rep < (kTopkBC * kTopkKC / 4) / kTopkThreads; ++rep) {
                const uint32_t f = tid + rep * kTopkThreads;
                const uint32_t row = f / (kTopkKC / 4), kq = f % (kTopkKC / 4);
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (c0 + row < nc && k0 + 4 * kq < d)
                    x = __ldcg(reinterpret_cast<const float4 *>(p.table) + (size_t)(p.cand_lo + c0 + row) * p.ld4 +
                               (k0 / 4 + kq));
                float *dst = Cs + (4 * kq) * (kTopkBC + kTopkPad) + row;
                dst[0] = x.x; dst[kTopkBC + kTopkPad] = x.y;
                dst[2 * (kTopkBC + kTopkPad)] = x.z; dst[3 * (kTopkBC + kTopkPad)] = x.w;
            }
            __syncthreads();
            const uint32_t kn = d - k0 < (uint32_t)kTopkKC ? d - k0 : (uint32_t)kTopkKC;
            for (uint32_t k = 0; k < kn; ++k) {
                float qv[TQ];
#pragma unroll
                for (int a = 0; a < TQ; ++a) qv[a] = Qs[(k0 + k) * BQ + ty * TQ + a];
                const float4 c_lo = *reinterpret_cast<const float4 *>(Cs + k * (kTopkBC + kTopkPad) + tx * 8);
                const float4 c_hi = *reinterpret_cast<const float4 *>(Cs + k * (kTopkBC + kTopkPad) + tx * 8 + 4);
                const float cv[8] = {c_lo.x, c_lo.y, c_lo.z, c_lo.w, c_hi.x, c_hi.y, c_hi.z, c_hi.w};
#pragma unroll
                for (int a = 0; a < TQ; ++a)
#pragma unroll
                    for (int b = 0; b < 8; ++b) acc[a][b] = fmaf(qv[a], cv[b], acc[a][b]);
            }
        }
        // ---- cosines; offer what can still enter a list, one candidate column per round ----
        float inv_c[8];
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const uint64_t c = c0 + tx * 8 + b;
            inv_c[b] = c < nc ? p.inv_norm[c] : 0.f;
        }
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const uint64_t c = c0 + tx * 8 + b;
            const long long cid = (long long)(p.cand_lo + c);
            int pushed = 0;
#pragma unroll
            for (int a = 0; a < TQ; ++a) {
                const uint32_t i = ty * TQ + a;
                const float cs = acc[a][b] * qinv[i] * inv_c[b];
                if (c < nc && qrow[i] >= 0 && cid != qrow[i] && cs > p.tau && (have[i] < p.K || cs >= thr[i])) {
                    const uint32_t slot = atomicAdd(&npush[i], 1u);      // < 16: one offer per tx thread
                    push_c[i * kTopkPush + slot] = cs;
                    push_i[i * kTopkPush + slot] = cid;
                    pushed = 1;
                }
            }
            if (__syncthreads_or(pushed)) {
                for (uint32_t i = wid; i < (uint32_t)BQ; i += kTopkThreads / 32) {
                    const uint32_t np = npush[i];
                    if (np == 0) continue;
                    uint32_t hv = have[i];
                    for (uint32_t s = 0; s < np; ++s)
                        list_insert(list_sc + (size_t)i * p.K, list_id + (size_t)i * p.K, hv, p.K,
                                    push_c[i * kTopkPush + s], push_i[i * kTopkPush + s], lane);
                    if (lane == 0) {
                        have[i] = hv; npush[i] = 0;
                        thr[i] = hv == p.K ? list_sc[(size_t)i * p.K + p.K - 1] : p.tau;
                    }
                }
                __syncthreads();
            }
        }
    }
    // ---- this block's lists out (padded with -1 / 0) ----
    __syncthreads();
    for (uint32_t e = tid; e < (uint32_t)BQ * p.K; e += kTopkThreads) {
        const uint32_t i = e / p.K, s = e % p.K;
        if (q0 + i >= p.m) continue;
        const size_t o = ((size_t)blockIdx.y * p.m + q0 + i) * p.K + s;
        const bool on = s < have[i];
        p.part_cos[o] = on ? list_sc[(size_t)i * p.K + s] : 0.f;
        p.part_ids[o] = on ? list_id[(size_t)i * p.K + s] : -1;
    }
}

// Merge the `splits` partial lists of each query: one warp per query.
__global__ void __launch_bounds__(kBlock)
topk_merge_kernel(const float *__restrict__ part_cos, const long long *__restrict__ part_ids, uint64_t m,
                  uint32_t K, uint32_t splits, float *__restrict__ out_cos, long long *__restrict__ out_ids)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    long long *id = reinterpret_cast<long long *>(smem_raw) + (size_t)wib * K;
    float *sc = reinterpret_cast<float *>(reinterpret_cast<long long *>(smem_raw) + (size_t)(blockDim.x >> 5) * K) +
                (size_t)wib * K;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t q = warp; q < m; q += nwarps) {
        uint32_t have = 0;
        for (uint32_t sp = 0; sp < splits; ++sp) {
            const size_t base = ((size_t)sp * m + q) * K;
            for (uint32_t s = 0; s < K; ++s) {
                const long long cid = part_ids[base + s];
                if (cid < 0) break;                               // lists are sorted and padded at the end
                list_insert(sc, id, have, K, part_cos[base + s], cid, lane);
            }
        }
        __syncwarp();
        for (uint32_t s = lane; s < K; s += 32) {
            out_cos[q * K + s] = s < have ? sc[s] : 0.f;
            out_ids[q * K + s] = s < have ? id[s] : -1;
        }
        __syncwarp();
    }
}

// ---- launchers --------------------------------------------------------------------------------
size_t topk_smem_bytes(uint32_t d, uint32_t K, int BQ)
{
    size_t b = (size_t)d * BQ * 4 + (size_t)kTopkKC * (kTopkBC + kTopkPad) * 4;     // Qs, Cs
    b += (size_t)BQ * K * 8 + (size_t)BQ * kTopkPush * 8 + (size_t)BQ * 8;          // list_id, push_i, qrow
    b += (size_t)BQ * K * 4 + (size_t)BQ * kTopkPush * 4 + (size_t)BQ * 4 * 4;      // list_sc, push_c, qinv/thr/have/npush
    return b;
}

int launch_inv_norms(const float *table, uint32_t d, uint32_t ld, uint64_t lo, uint64_t count, float *inv_norm,
                     int sms, cudaStream_t s)
{
    if (count == 0) return 0;
    const uint64_t want = (count + (kBlock / 32) - 1) / (kBlock / 32);
    const int grid = (int)(want < (uint64_t)sms * 8 ? want : (uint64_t)sms * 8);
    row_inv_norm_kernel<<<grid, kBlock, 0, s>>>(table, d / 4, ld / 4, lo, count, inv_norm);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

// Returns launches made, -1 on a launch error, -2 if the shape does not fit shared memory.
int launch_topk(const float *table, uint32_t d, uint32_t ld, uint64_t vocab, const long long *queries, uint64_t m,
                uint64_t cand_lo, uint64_t cand_hi, uint32_t K, float tau, const float *inv_norm, float *part_cos,
                long long *part_ids, uint32_t splits, float *out_cos, long long *out_ids, int sms, cudaStream_t s)
{
    if (m == 0) return 0;
    TopkParams p;
    p.table = table; p.queries = queries; p.inv_norm = inv_norm;
    p.part_cos = splits > 1 ? part_cos : out_cos; p.part_ids = splits > 1 ? part_ids : out_ids;
    p.m = m; p.vocab = vocab; p.cand_lo = cand_lo; p.cand_hi = cand_hi;
    p.d4 = d / 4; p.ld4 = ld / 4; p.K = K; p.splits = splits; p.tau = tau;
    const size_t limit = 227 * 1024;
    int launched = 0;
    if (topk_smem_bytes(d, K, 64) <= limit) {
        const size_t sm = topk_smem_bytes(d, K, 64);
        if (cudaFuncSetAttribute(topk_cosine_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess)
            return -1;
        dim3 grid((unsigned)((m + 63) / 64), splits);
        topk_cosine_kernel<64><<<grid, kTopkThreads, sm, s>>>(p);
    } else if (topk_smem_bytes(d, K, 32) <= limit) {
        const size_t sm = topk_smem_bytes(d, K, 32);
        if (cudaFuncSetAttribute(topk_cosine_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess)
            return -1;
        dim3 grid((unsigned)((m + 31) / 32), splits);
        topk_cosine_kernel<32><<<grid, kTopkThreads, sm, s>>>(p);
    } else {
        return -2;
    }
    if (cudaGetLastError() != cudaSuccess) return -1;
    ++launched;
    if (splits > 1) {
        const int warps = kBlock / 32;
        const uint64_t want = (m + warps - 1) / warps;
        const int grid = (int)(want < (uint64_t)sms * 8 ? want : (uint64_t)sms * 8);
        topk_merge_kernel<<<grid, kBlock, (size_t)warps * K * 12, s>>>(part_cos, part_ids, m, K, splits, out_cos, out_ids);
        if (cudaGetLastError() != cudaSuccess) return -1;
        ++launched;
    }
    (void)sms;
    return launched;
}

}  // namespace w2v

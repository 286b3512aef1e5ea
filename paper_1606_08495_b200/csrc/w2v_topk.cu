// Retrieval by cosine similarity over the trained vectors (Section 2: "calculating cosine
// similarity between the ad vector and all query vectors.  The K queries with the highest
// similarity are retrieved"; Section 7.2: K = 30 nearest, kept only above tau = 0.65).
//
// For a block of BQ query rows the kernel streams the candidate rows in tiles of BC, forms the
// BQ x BC dot products in registers (a 16 x 32 thread grid, each thread (BQ/16) x 8 of them; both
// operands staged through shared memory, k-major), scales them by the inverse norms and feeds the
// ones that can still enter a query's list into that query's sorted top-K list in shared memory.
// All arithmetic is fp32 on the CUDA cores: cosines agree with a double-precision evaluation to
// ~1e-6.  (w2v_topk_tc.cu is the tensor-core kernel for the same contract; this one is selected with
// w2v_set_retrieval_kernel(h, 0).)  The merge kernel and the split plan below serve both.
#include "w2v_device.cuh"
#include "w2v_internal.h"

namespace w2v {

constexpr int kTopkBC = 256;          // candidate rows per tile
constexpr int kTopkKC = 16;           // columns per shared-memory chunk
constexpr int kTopkPad = 4;           // keeps 16-byte alignment of the k-major rows
constexpr int kTopkThreads = 512;     // 16 query groups x 32 candidate groups
constexpr int kTopkTX = 32;           // threads along the candidates
constexpr int kTopkPush = kTopkTX;    // at most one offer per candidate thread to a query per round

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
    // layout: Qs[nch*KC][BQ] | Cs[2][KC][BC+pad] | list_sc[BQ][K] | list_id[BQ][K] | push_c[BQ][16] | push_i[BQ][16]
    //         | qinv[BQ] | thr[BQ] | have[BQ] | npush[BQ] | qrow[BQ]
    const uint32_t nch = (d + kTopkKC - 1) / kTopkKC;       // column chunks; Qs is zero-padded to nch * KC rows
    float *Qs = reinterpret_cast<float *>(smem_raw);
    float *Cs = Qs + (size_t)nch * kTopkKC * BQ;            // two buffers of KC x (BC + pad)
    constexpr int kCsBuf = kTopkKC * (kTopkBC + kTopkPad);
    long long *list_id = reinterpret_cast<long long *>(Cs + 2 * kCsBuf);
    long long *push_i = list_id + (size_t)BQ * p.K;
    long long *qrow = push_i + BQ * kTopkPush;
    float *list_sc = reinterpret_cast<float *>(qrow + BQ);
    float *push_c = list_sc + (size_t)BQ * p.K;
    float *qinv = push_c + BQ * kTopkPush;
    float *thr = qinv + BQ;
    uint32_t *have = reinterpret_cast<uint32_t *>(thr + BQ);
    uint32_t *npush = have + BQ;

    const uint32_t tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint32_t tx = tid & (kTopkTX - 1), ty = tid / kTopkTX;
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
    for (uint32_t e = d * BQ + tid; e < nch * kTopkKC * BQ; e += kTopkThreads) Qs[e] = 0.f;
    __syncthreads();
    for (uint32_t i = wid; i < (uint32_t)BQ; i += kTopkThreads / 32) {
        float s = 0.f;
        for (uint32_t k = lane; k < d; k += 32) s = fmaf(Qs[k * BQ + i], Qs[k * BQ + i], s);
        s = warp_sum(s);
        if (lane == 0) qinv[i] = s > 0.f ? 1.0f / sqrtf(s) : 0.f;
    }
    __syncthreads();

    // Candidate columns are staged chunk by chunk (KC columns of BC rows, transposed); the global
    // loads of chunk g+1 are in flight while chunk g is multiplied.
    constexpr int kRep = (kTopkBC * kTopkKC / 4) / kTopkThreads;
    const uint64_t total_g = (t_hi - t_lo) * nch;
    auto gload = [&](uint64_t tile, uint32_t chunk, float4 (&x)[kRep]) {
        const uint64_t c0 = tile * kTopkBC;
        const uint32_t k0 = chunk * kTopkKC;
#pragma unroll
        for (int rep = 0; rep < kRep; ++rep) {
            const uint32_t f = tid + rep * kTopkThreads;
            const uint32_t row = f / (kTopkKC / 4), kq = f % (kTopkKC / 4);
            x[rep] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c0 + row < nc && k0 + 4 * kq < d)
                x[rep] = __ldcg(reinterpret_cast<const float4 *>(p.table) + (size_t)(p.cand_lo + c0 + row) * p.ld4 +
                                (k0 / 4 + kq));
        }
    };
    auto sstore = [&](float *buf, const float4 (&x)[kRep]) {
#pragma unroll
        for (int rep = 0; rep < kRep; ++rep) {
            const uint32_t f = tid + rep * kTopkThreads;
            const uint32_t row = f / (kTopkKC / 4), kq = f % (kTopkKC / 4);
            float *dst = buf + (4 * kq) * (kTopkBC + kTopkPad) + row;
            dst[0] = x[rep].x; dst[kTopkBC + kTopkPad] = x[rep].y;
            dst[2 * (kTopkBC + kTopkPad)] = x[rep].z; dst[3 * (kTopkBC + kTopkPad)] = x[rep].w;
        }
    };
    float acc[TQ][8];
    {
        float4 x0[kRep];
        if (total_g) { gload(t_lo, 0, x0); sstore(Cs, x0); }
    }
    __syncthreads();
    uint64_t tile = t_lo;
    uint32_t chunk = 0;
    for (uint64_t g = 0; g < total_g; ++g, ++chunk) {
        if (chunk == nch) { chunk = 0; ++tile; }
        const uint64_t c0 = tile * kTopkBC;                      // first candidate of the tile (relative)
        const float *cbuf = Cs + (g & 1) * kCsBuf;
        float4 xn[kRep];
        const bool more = g + 1 < total_g;
        if (more) gload(chunk + 1 == nch ? tile + 1 : tile, chunk + 1 == nch ? 0u : chunk + 1, xn);
        if (chunk == 0) {
#pragma unroll
            for (int a = 0; a < TQ; ++a)
#pragma unroll
                for (int b = 0; b < 8; ++b) acc[a][b] = 0.f;
        }
        const float *qbase = Qs + (size_t)chunk * kTopkKC * BQ + ty * TQ;
#pragma unroll
        for (int k = 0; k < kTopkKC; ++k) {
            float qv[TQ];
            if constexpr (TQ == 4) {
                const float4 q4 = *reinterpret_cast<const float4 *>(qbase + k * BQ);
                qv[0] = q4.x; qv[1] = q4.y; qv[2] = q4.z; qv[3] = q4.w;
            } else {
#pragma unroll
                for (int a = 0; a < TQ; ++a) qv[a] = qbase[k * BQ + a];
            }
            // a thread's 8 candidates are columns 4 tx .. 4 tx + 3 and BC/2 + 4 tx .. : the threads
            // of a warp read 512 contiguous bytes per load, without bank conflicts
            const float4 c_lo = *reinterpret_cast<const float4 *>(cbuf + k * (kTopkBC + kTopkPad) + tx * 4);
            const float4 c_hi = *reinterpret_cast<const float4 *>(cbuf + k * (kTopkBC + kTopkPad) + kTopkBC / 2 + tx * 4);
            const float cv[8] = {c_lo.x, c_lo.y, c_lo.z, c_lo.w, c_hi.x, c_hi.y, c_hi.z, c_hi.w};
#pragma unroll
            for (int a = 0; a < TQ; ++a)
#pragma unroll
                for (int b = 0; b < 8; ++b) acc[a][b] = fmaf(qv[a], cv[b], acc[a][b]);
        }
        if (more) sstore(Cs + ((g + 1) & 1) * kCsBuf, xn);
        __syncthreads();
        if (chunk != nch - 1) continue;
        // ---- cosines; offer what can still enter a list, one candidate column per round ----
        float inv_c[8];
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const uint64_t c = c0 + (b < 4 ? tx * 4 + b : kTopkBC / 2 + tx * 4 + (b - 4));
            inv_c[b] = c < nc ? p.inv_norm[c] : 0.f;
        }
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const uint64_t c = c0 + (b < 4 ? tx * 4 + b : kTopkBC / 2 + tx * 4 + (b - 4));
            const long long cid = (long long)(p.cand_lo + c);
            int pushed = 0;
#pragma unroll
            for (int a = 0; a < TQ; ++a) {
                const uint32_t i = ty * TQ + a;
                const float cs = acc[a][b] * qinv[i] * inv_c[b];
                if (c < nc && qrow[i] >= 0 && cid != qrow[i] && cs > p.tau && (have[i] < p.K || cs >= thr[i])) {
                    const uint32_t slot = atomicAdd(&npush[i], 1u);      // < kTopkPush: one offer per tx thread
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
    const size_t nch = (d + kTopkKC - 1) / kTopkKC;
    size_t b = nch * kTopkKC * BQ * 4 + 2 * (size_t)kTopkKC * (kTopkBC + kTopkPad) * 4;  // Qs (padded), two Cs
    b += (size_t)BQ * K * 8 + (size_t)BQ * kTopkPush * 8 + (size_t)BQ * 8;          // list_id, push_i, qrow
    b += (size_t)BQ * K * 4 + (size_t)BQ * kTopkPush * 4 + (size_t)BQ * 4 * 4;      // list_sc, push_c, qinv/thr/have/npush
    return b;
}

// How many ways to split the candidates so that the grid fills whole waves of one block per SM:
// the smallest split count (at most 64, at most one per tile) whose last wave is at least `min_fill`
// full (95 % unless given), else the fullest one.
uint32_t topk_splits(uint64_t m, uint64_t n_candidates, int sms, uint32_t block_queries, uint32_t tile_rows, double min_fill)
{
    if (block_queries == 0) { block_queries = 64; tile_rows = kTopkBC; }
    const uint64_t qblocks = (m + block_queries - 1) / block_queries, tiles = (n_candidates + tile_rows - 1) / tile_rows;
    uint64_t max_s = tiles < 64 ? (tiles ? tiles : 1) : 64;
    uint32_t best = 1;
    double best_fill = 0.0;
    for (uint64_t sp = 1; sp <= max_s; ++sp) {
        const uint64_t blocks = qblocks * sp, waves = (blocks + sms - 1) / sms;
        const double fill = (double)blocks / (double)(waves * sms);
        if (fill > best_fill + 1e-9) { best_fill = fill; best = (uint32_t)sp; }
        if (fill >= min_fill) return (uint32_t)sp;
    }
    return best;
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

int launch_topk_merge(const float *part_cos, const long long *part_ids, uint64_t m, uint32_t K, uint32_t splits,
                      float *out_cos, long long *out_ids, int sms, cudaStream_t s)
{
    if (m == 0) return 0;
    const int warps = kBlock / 32;
    const uint64_t want = (m + warps - 1) / warps;
    const int grid = (int)(want < (uint64_t)sms * 8 ? want : (uint64_t)sms * 8);
    topk_merge_kernel<<<grid, kBlock, (size_t)warps * K * 12, s>>>(part_cos, part_ids, m, K, splits, out_cos, out_ids);
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

// Cosine retrieval on the tensor cores (tcgen05, TMEM accumulators), same contract as the fp32
// kernel in w2v_topk.cu.  Two kernels: first the one that forms every cosine to full accuracy on the
// tensor cores (three TF32 MMAs per product), then, further down, the default: a bf16 screen followed
// by exact fp32 cosines for the few candidates that the screen cannot dismiss.
//
// The dot products of 128 query rows with 256 candidate rows are one M128 x N256 accumulator tile in
// tensor memory.  The tensor cores read fp32 operands as TF32 (the 13 low mantissa bits are
// ignored), which alone would leave cosines good to 1e-3 only; the threshold and the ranking need
// 1e-6.  So every value x is split into hi = x rounded to TF32 and lo = (x - hi) rounded to TF32, and
// each k-step issues three MMAs into the same accumulator: lo.hi + hi.lo + hi.hi (the dropped lo.lo
// term and the rounding of lo are below 2^-21 of |a||b| and unbiased).
//
// One block = 416 threads:
//   warps 0-3  epilogue: warp w reads accumulator rows 32w .. 32w+31 (thread = one query) from
//              tensor memory, scales by the inverse norms and keeps that query's sorted top-K list;
//   warp 4     allocates tensor memory; one lane issues the MMAs;
//   warps 5-12 loaders (two groups of 4 warps, one per stage of the ring): candidate rows -> (hi, lo) -> shared memory
//              (the query side is split once by a pre-pass and arrives by cp.async.bulk), K-major core-matrix layout without
//              swizzle ([16-byte column chunk][row][16 B], chunk stride 2064 B: conflict-free stores).
// Shared-memory stages and the two accumulator buffers are handed over with mbarriers; every wait
// has a time limit, after which the block raises the error flag and leaves through the common
// exit that frees the tensor memory.
#include "w2v_device.cuh"
#include "w2v_internal.h"

namespace w2v {

constexpr int kTcM = 128;                       // query rows per block (accumulator lanes)
constexpr int kTcN = 256;                       // candidate rows per tile (accumulator columns)
constexpr int kTcKB = 32;                       // floats per K-block = 8 chunks of 16 B = 4 MMAs of K = 8
constexpr int kTcStages = 2;
constexpr int kTcChunkStride = kTcM * 16 + 16;  // bytes between 16-byte column chunks of a query operand
constexpr int kTcOperand = 8 * kTcChunkStride;  // bytes of one query operand block (128 rows x 32 floats)
constexpr int kTcChunkStrideC = kTcN * 16 + 16; // the same for a candidate operand (256 rows)
constexpr int kTcOperandC = 8 * kTcChunkStrideC;
constexpr int kTcStageBytes = 2 * kTcOperand + 2 * kTcOperandC;   // Q hi, Q lo, C hi, C lo
constexpr int kTcLoaders = 128;                 // threads that fill one stage together
constexpr int kTcGroups = 2;                    // loader groups; group j fills stages j, j + 2, ...
constexpr int kTcThreads = 5 * 32 + kTcGroups * kTcLoaders;
constexpr uint32_t kTcSpinLimit = 1u << 20;

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return done != 0;
}
// Bounded wait.  Returns false (and raises the block's abort flag) when the limit is reached or
// another thread has already given up.  The limit is a time, not a count: how long a partner may
// legitimately take depends on the data (an epilogue warp computes an exact cosine for every pair
// that passes the screen, which for rows that are all alike is every pair).
constexpr unsigned long long kTcWaitNs = 4000000000ull;           // 4 s
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                          unsigned long long limit_ns = kTcWaitNs)
{
    unsigned long long t0 = 0;                                      // the clock is read only by a wait that lasts
    for (uint32_t spin = 0; spin < (1u << 30); ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 1023u) == 1023u) {
            if (*abort_flag) return false;
            if (!t0) t0 = global_ns();
            else if (global_ns() - t0 > limit_ns) break;
        }
    }
    *abort_flag = 1;
    return false;
}

// Shared-memory matrix descriptor: K-major, no swizzle; 8 rows x 16 B core matrices, `lbo` bytes
// between the two 16-byte column chunks of one MMA, `sbo` bytes between groups of 8 rows.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0), "r"(0), "r"(0), "r"(0) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// Does (score a, id ia) rank ahead of (score b, id ib)?  Larger cosine first, then smaller id.
__device__ __forceinline__ bool ranks_ahead_tc(float a, long long ia, float b, long long ib)
{
    return a > b || (a == b && ia < ib);
}

// One candidate for a thread's own sorted list (in global memory, private to the thread).
__device__ __noinline__ void list_offer(float *lc, long long *li, uint32_t &have, float &thr, uint32_t K, float tau,
                                        float cs, long long cid, long long self)
{
    if (!(cs > tau) || cid == self || (have == K && cs < thr)) return;
    uint32_t pos = have;
    while (pos > 0 && ranks_ahead_tc(cs, cid, lc[pos - 1], li[pos - 1])) --pos;
    if (pos >= K) return;
    const uint32_t last = have < K ? have : K - 1u;
    for (uint32_t s = last; s > pos; --s) { lc[s] = lc[s - 1]; li[s] = li[s - 1]; }
    lc[pos] = cs; li[pos] = cid;
    if (have < K) ++have;
    thr = have == K ? lc[K - 1] : tau;
}

struct TcParams {
    const float *table;
    const long long *queries;
    const float *inv_norm;
    const unsigned char *qsplit;  // [query blocks][K-blocks][hi, lo] operand blocks, laid out as in shared memory
    const unsigned char *ctiles;  // screening kernel: candidate operand blocks (topk_pack_candidates_kernel)
    unsigned int *floor_q;        // screening kernel: [m] best K-th cosine any block has reached for the query (ordered encoding, 0 = none)
    float *part_cos;              // [splits][m][K]
    long long *part_ids;
    int *error;                   // device word: set to 1 if a wait ran out
    uint64_t m, vocab, cand_lo, cand_hi;
    uint32_t d4, ld4, K, splits;
    float tau;
};

// x rounded to the nearest value with 10 explicit mantissa bits (ties away from zero), so that the
// tensor core, which drops the 13 low bits, reads it exactly.
__device__ __forceinline__ float tf32_round(float x)
{
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);
}

__device__ __forceinline__ void split_store(unsigned char *hi, unsigned char *lo, uint32_t r, uint32_t ch, float4 v,
                                            uint32_t chunk_stride)
{
    const float4 h = make_float4(tf32_round(v.x), tf32_round(v.y), tf32_round(v.z), tf32_round(v.w));
    const float4 l = make_float4(tf32_round(v.x - h.x), tf32_round(v.y - h.y), tf32_round(v.z - h.z),
                                 tf32_round(v.w - h.w));
    const uint32_t off = ch * chunk_stride + r * 16;
    *reinterpret_cast<float4 *>(hi + off) = h;
    *reinterpret_cast<float4 *>(lo + off) = l;
}

// The query side is the same for every candidate tile: it is split once, into global scratch that
// has the layout of the shared-memory operand blocks, and the main kernel copies it in bulk.
// One block per (query block, K-block).
__global__ void __launch_bounds__(256)
topk_split_queries_kernel(const float *__restrict__ table, const long long *__restrict__ queries, uint64_t m,
                          uint64_t vocab, uint32_t d4, uint32_t ld4, uint32_t nkb, unsigned char *__restrict__ qsplit)
{
    const uint32_t qb = blockIdx.x / nkb, kb = blockIdx.x % nkb;
    unsigned char *hi = qsplit + ((size_t)qb * nkb + kb) * 2 * kTcOperand, *lo = hi + kTcOperand;
    const float4 *T4 = reinterpret_cast<const float4 *>(table);
    for (uint32_t e = threadIdx.x; e < (uint32_t)kTcM * 8; e += blockDim.x) {
        const uint32_t r = e >> 3, ch = e & 7;
        const uint64_t qi = (uint64_t)qb * kTcM + r;
        long long row = qi < m ? queries[qi] : -1;
        if (row < 0 || (unsigned long long)row >= vocab) row = -1;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row >= 0 && kb * 8 + ch < d4) x = __ldcg(T4 + (size_t)row * ld4 + (kb * 8 + ch));
        split_store(hi, lo, r, ch, x, kTcChunkStride);
    }
    // the 16 padding bytes at the end of each chunk are copied too: keep them defined
    if (threadIdx.x < 8) {
        *reinterpret_cast<float4 *>(hi + threadIdx.x * kTcChunkStride + kTcM * 16) = make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4 *>(lo + threadIdx.x * kTcChunkStride + kTcM * 16) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

// One stage of candidates: 128 rows x 32 floats of the table -> (hi, lo) operand blocks, in two
// halves so that the global loads can be issued before the stage's slot in shared memory is free.
constexpr int kTcPer = (kTcN * 8) / kTcLoaders;                  // float4 per loader thread and stage

__device__ __forceinline__ void candidates_issue(const TcParams &p, float4 (&x)[kTcPer], uint32_t k0, uint32_t ltid,
                                                 uint64_t c0, uint64_t nc)
{
    const float4 *T4 = reinterpret_cast<const float4 *>(p.table);
#pragma unroll
    for (int it = 0; it < kTcPer; ++it) {
        const uint32_t e = ltid + it * kTcLoaders;
        const uint32_t r = e >> 3, ch = e & 7;                   // 8 threads cover 128 contiguous bytes of a row
        x[it] = (c0 + r < nc && k0 / 4 + ch < p.d4) ? __ldcg(T4 + (size_t)(p.cand_lo + c0 + r) * p.ld4 + (k0 / 4 + ch))
                                                    : make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

__device__ __forceinline__ void candidates_store(unsigned char *hi, unsigned char *lo, const float4 (&x)[kTcPer],
                                                 uint32_t ltid)
{
#pragma unroll
    for (int it = 0; it < kTcPer; ++it) {
        const uint32_t e = ltid + it * kTcLoaders;
        split_store(hi, lo, e >> 3, e & 7, x[it], kTcChunkStrideC);
    }
}

__device__ __forceinline__ void bulk_to_smem(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

__global__ void __launch_bounds__(kTcThreads, 1)
topk_cosine_tc_kernel(TcParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + kTcStages * kTcStageBytes);
    uint64_t *empty = full + kTcStages;
    uint64_t *tfull = empty + kTcStages;
    uint64_t *tempty = tfull + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tempty + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    long long *qrow = reinterpret_cast<long long *>(tmem_slot + 4);          // [128]
    float *inv_c = reinterpret_cast<float *>(qrow + kTcM);                   // [4 warps][2][kTcN]

    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint64_t q0 = (uint64_t)blockIdx.x * kTcM;
    const uint64_t nc = p.cand_hi - p.cand_lo;
    const uint64_t tiles = (nc + kTcN - 1) / kTcN;
    const uint64_t t_lo = tiles * blockIdx.y / p.splits, t_hi = tiles * (blockIdx.y + 1) / p.splits;
    const uint32_t d = 4u * p.d4;
    const uint32_t nkb = (d + kTcKB - 1) / kTcKB;
    const uint64_t n_tiles = t_hi - t_lo;

    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) { mbar_init(full + s, kTcLoaders); mbar_init(empty + s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull + b, 1); mbar_init(tempty + b, kTcM); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < (uint32_t)kTcM) {
        long long r = q0 + tid < p.m ? p.queries[q0 + tid] : -1;
        if (r < 0 || (unsigned long long)r >= p.vocab) r = -1;
        qrow[tid] = r;
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)), "r"(2 * kTcN));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4) {
        // ================= epilogue: one thread per query row =================
        const uint32_t r = tid;
        const long long my_q = qrow[r];
        const bool live = q0 + r < p.m;
        float *lc = p.part_cos + ((size_t)blockIdx.y * p.m + (q0 + r)) * p.K;      // this query's list (global, private)
        long long *li = p.part_ids + ((size_t)blockIdx.y * p.m + (q0 + r)) * p.K;
        float qinv = 0.f;
        if (my_q >= 0) {
            const float4 *row = reinterpret_cast<const float4 *>(p.table) + (size_t)my_q * p.ld4;
            float s = 0.f;
            for (uint32_t j = 0; j < p.d4; ++j) {
                const float4 x = __ldcg(row + j);
                s = fmaf(x.x, x.x, s); s = fmaf(x.y, x.y, s); s = fmaf(x.z, x.z, s); s = fmaf(x.w, x.w, s);
            }
            qinv = s > 0.f ? 1.0f / sqrtf(s) : 0.f;
        }
        if (live) for (uint32_t s = 0; s < p.K; ++s) { lc[s] = 0.f; li[s] = -1; }
        uint32_t have = 0;
        float thr = p.tau;
        for (uint64_t i = 0; i < n_tiles; ++i) {
            const uint32_t b = (uint32_t)(i & 1);
            const uint64_t c0 = (t_lo + i) * kTcN;
            // inverse norms of the tile's candidates (0 past the end of the range), staged in shared
            // memory while the tile's MMAs are still running
            float *icn = inv_c + (warp * 2 + b) * kTcN;             // one copy per warp: no block-wide barrier here
            for (uint32_t j = lane; j < (uint32_t)kTcN; j += 32) icn[j] = c0 + j < nc ? __ldg(p.inv_norm + c0 + j) : 0.f;
            __syncwarp();
            // the tensor-memory loads below are warp-wide: the whole warp goes on or gives up together
            if (!__all_sync(kFullMask, mbar_wait(tfull + b, (uint32_t)((i >> 1) & 1), abort_flag))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const bool mine = my_q >= 0 && live;
#pragma unroll 1
            for (uint32_t cc = 0; cc < (uint32_t)kTcN; cc += 32) {
                uint32_t v[32];
                __syncwarp();
                const uint32_t ta = tmem_base + ((warp * 32u) << 16) + b * kTcN + cc;
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                             "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                             "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                             : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                               "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                               "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                               "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                             : "r"(ta));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (!mine) continue;
                // fast filter: which of the 32 cosines reach the current cut at all?
                float cut = have < p.K ? p.tau : fmaxf(p.tau, thr);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float cs = __uint_as_float(v[j]) * qinv * icn[cc + j];
                    if (cs >= cut) {                               // rare: exact test and sorted insertion
                        const uint64_t c = c0 + cc + j;
                        if (c < nc) list_offer(lc, li, have, thr, p.K, p.tau, cs, (long long)(p.cand_lo + c), my_q);
                        cut = have < p.K ? p.tau : fmaxf(p.tau, thr);
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(tempty + b);                              // this accumulator buffer may be overwritten
        }
    } else if (warp == 4) {
        // ================= MMA issue: one lane =================
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(kTcN >> 3) << 17) | ((uint32_t)(kTcM >> 4) << 24);
            uint64_t g = 0;
            bool ok = true;
            for (uint64_t i = 0; i < n_tiles && ok; ++i) {
                const uint32_t b = (uint32_t)(i & 1);
                ok = mbar_wait(tempty + b, (uint32_t)(((i >> 1) & 1) ^ 1), abort_flag);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t dst = tmem_base + b * kTcN;
                for (uint32_t kb = 0; kb < nkb && ok; ++kb, ++g) {
                    const uint32_t s = (uint32_t)(g % kTcStages);
                    ok = mbar_wait(full + s, (uint32_t)((g / kTcStages) & 1), abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t base = smem_addr(smem + (size_t)s * kTcStageBytes);
#pragma unroll
                    for (int kk = 0; kk < kTcKB / 8; ++kk) {
                        const uint32_t off = 2 * kk * kTcChunkStride, offc = 2 * kk * kTcChunkStrideC;
                        const uint64_t qh = umma_desc(base + 0 * kTcOperand + off, kTcChunkStride, 128);
                        const uint64_t ql = umma_desc(base + 1 * kTcOperand + off, kTcChunkStride, 128);
                        const uint64_t ch = umma_desc(base + 2 * kTcOperand + offc, kTcChunkStrideC, 128);
                        const uint64_t cl = umma_desc(base + 2 * kTcOperand + kTcOperandC + offc, kTcChunkStrideC, 128);
                        umma_tf32(dst, ql, ch, idesc, (kb | kk) ? 1u : 0u);      // small terms first
                        umma_tf32(dst, qh, cl, idesc, 1u);
                        umma_tf32(dst, qh, ch, idesc, 1u);
                    }
                    umma_commit(empty + s);                       // the stage is free once these MMAs have read it
                }
                if (ok) umma_commit(tfull + b);                   // the tile's accumulator is complete
            }
        }
    } else {
        // ================= loaders =================
        // group j fills stages j, j + kTcGroups, ...; the loads of a stage are issued before its slot
        // is waited for, so they overlap the MMAs that still read the slot
        const uint32_t group = (tid - 5 * 32) / kTcLoaders, ltid = (tid - 5 * 32) % kTcLoaders;
        const uint64_t total_g = n_tiles * nkb;
        float4 x[kTcPer];
        uint64_t g = group;
        if (g < total_g) candidates_issue(p, x, (uint32_t)(g % nkb) * kTcKB, ltid, (t_lo + g / nkb) * kTcN, nc);
        while (g < total_g) {
            const uint32_t s = (uint32_t)(g % kTcStages), kb = (uint32_t)(g % nkb);
            if (!mbar_wait(empty + s, (uint32_t)(((g / kTcStages) & 1) ^ 1), abort_flag)) break;
            unsigned char *st = smem + (size_t)s * kTcStageBytes;
            if (ltid == 0) {
                // the query side arrives by bulk copy; its bytes complete the same barrier
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                             ::"r"(smem_addr(full + s)), "r"(2u * kTcOperand) : "memory");
                bulk_to_smem(st, p.qsplit + ((size_t)blockIdx.x * nkb + kb) * 2 * kTcOperand, 2u * kTcOperand, full + s);
            }
            candidates_store(st + 2 * kTcOperand, st + 2 * kTcOperand + kTcOperandC, x, ltid);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");         // stores -> tensor-core reads
            if (ltid != 0) mbar_arrive(full + s);
            g += kTcGroups;
            if (g < total_g) candidates_issue(p, x, (uint32_t)(g % nkb) * kTcKB, ltid, (t_lo + g / nkb) * kTcN, nc);
        }
    }
    // ================= common exit =================
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0 && *abort_flag) atomicExch(p.error, 1);
    if (warp == 4) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kTcN));
    }
}

// =================================================================================================
// Screening variant.  One low-precision MMA per product instead of three TF32 ones: both sides are
// rounded to bf16 (8 significant bits: relative error at most 2^-8 per value), so each product is off
// by at most (2^-7 + 2^-16) |a_i b_i| and, by Cauchy-Schwarz, the cosine by less than 7.83e-3; the fp32
// accumulation adds some 1e-5.  (Rows of a few hundred columns come nowhere near: 6e-4 is typical at
// d = 300; rows of 4 columns reach 5e-3.)  That is enough to decide that a candidate cannot reach a
// query's current cut.  Only a candidate whose approximate cosine comes within kScreenEps of the cut is
// looked at again: its warp computes the fp32 dot product of the two rows from the table, and that
// exact cosine goes to the sorted list.  With a list of K the number of such candidates is about
// K ln(n / K) per query, against n screened.
//
// Both sides are converted by pre-passes into global scratch that has exactly the layout of the
// shared-memory operands ([K-block][16-byte chunk][row][8 bf16]), so the main kernel moves them
// with bulk copies only and has no loader warps.  The query block stays in shared memory for the
// whole kernel (d <= 320: 80 KB); candidates stream through three 48 KB stages (three K-blocks of 32
// columns of a 256-candidate tile: six MMAs of K = 16), each filled by one `cp.async.bulk` that a
// single producer lane issues as soon as the stage's previous MMAs have committed.  The stage is
// that large because one lane hands over a stage every 250-330 ns whatever its size (w2v_probe_bulk_ring:
// a ring of bulk copies alone, without MMAs, moves 50-66 GB/s per SM with 16 KB stages at any depth,
// twice that with 32 KB and three times with 48 KB stages): with 16 KB stages that hand-over rate, not
// bytes or MMAs, bounded the kernel (19.0 -> 16.6 ms for 8192 queries x 3 M candidates; 32 KB x 4 and
// 64 KB x 2 measure the same).  The next bound was what the MMA lane executes per MMA (16.6 -> 13.6 ms,
// see its loop), and every wait in that lane still costs tensor-pipe time.
constexpr float kScreenEps = 8.5e-3f;
constexpr int kScKB = 32;                                        // columns per stage
constexpr int kScCh = kScKB / 8;                                 // 16-byte chunks (8 bf16) per row and stage
constexpr int kScMaxKB = 10;                                     // K-blocks of a query block that can stay in shared memory: d <= 320
constexpr int kScStages = 3;
constexpr int kScKPS = 3;                                        // K-blocks per stage (consecutive K-blocks of a tile are contiguous in the packed copy)
constexpr int kScAChunk = kTcM * 16;                             // query operand, one 16-byte chunk of all rows
constexpr int kScABlock = kScCh * kScAChunk;                     // bytes of one K-block of the query operand
constexpr int kScBChunk = kTcN * 16;                             // candidate operand
constexpr int kScStageBytes = kScCh * kScBChunk;                 // one stage = one K-block of one candidate tile = one bulk copy
constexpr int kExact = 4;                                        // (query, candidate) pairs whose exact cosines are computed together
constexpr int kScThreads = 6 * 32;                               // 4 epilogue warps, the MMA warp, the producer warp

// two floats -> two bf16 (round to nearest even), first in the low half
__device__ __forceinline__ uint32_t bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Query rows of one block as bf16 in the layout of the shared-memory operand
// ([K-block][16-byte chunk][row][8 bf16]).  One block per (query block, K-block).
__global__ void __launch_bounds__(256)
topk_round_queries_kernel(const float *__restrict__ table, const long long *__restrict__ queries, uint64_t m,
                          uint64_t vocab, uint32_t d4, uint32_t ld4, uint32_t nkb, unsigned char *__restrict__ qb16)
{
    const uint32_t qb = blockIdx.x / nkb, kb = blockIdx.x % nkb;
    unsigned char *dst = qb16 + ((size_t)qb * nkb + kb) * kScABlock;
    const float4 *T4 = reinterpret_cast<const float4 *>(table);
    for (uint32_t e = threadIdx.x; e < (uint32_t)(kTcM * kScCh); e += blockDim.x) {
        const uint32_t r = e / kScCh, ch = e % kScCh;
        const uint64_t qi = (uint64_t)qb * kTcM + r;
        long long row = qi < m ? queries[qi] : -1;
        if (row < 0 || (unsigned long long)row >= vocab) row = -1;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
        const uint32_t c4 = kb * (kScKB / 4) + 2 * ch;                      // first of the two float4 of this chunk
        if (row >= 0 && c4 < d4) x = __ldcg(T4 + (size_t)row * ld4 + c4);
        if (row >= 0 && c4 + 1 < d4) y = __ldcg(T4 + (size_t)row * ld4 + c4 + 1);
        *reinterpret_cast<uint4 *>(dst + ch * kScAChunk + r * 16) =
            make_uint4(bf16x2(x.x, x.y), bf16x2(x.z, x.w), bf16x2(y.x, y.y), bf16x2(y.z, y.w));
    }
}

// Candidate rows cand_lo + [0, nc), scaled to unit length, as bf16 operand blocks:
// [tile of NT rows][K-block][chunk][row][8 bf16] for `tiles` tiles, zeros past the end of the range and of
// the row (NT = 256 for the one-block kernel, 128 for the pair kernel, whose blocks take a half tile each);
// inv_norm[c] = 1/|row c| (0 for a zero row) is written on the way, for the exact cosines.
// One block per tile, one thread per row: a thread reads its row once for the norm and once more,
// 128 bytes (one K-block) at a time through L1 and L2, for the operand; the NT threads' 16-byte
// stores of one chunk are contiguous.
template <int NT>
__global__ void __launch_bounds__(NT)
topk_pack_candidates_kernel(const float *__restrict__ table, float *__restrict__ inv_norm, uint32_t d4, uint32_t ld4,
                            uint64_t cand_lo, uint64_t nc, uint64_t tiles, uint32_t nkb, unsigned char *__restrict__ out)
{
    constexpr int kBChunk = NT * 16, kBStage = kScCh * kBChunk;
    const uint32_t r = threadIdx.x;
    for (uint64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const uint64_t c = tile * NT + r;
        const bool valid = c < nc;
        const float4 *row = reinterpret_cast<const float4 *>(table) + (size_t)(cand_lo + (valid ? c : 0)) * ld4;
        float ic = 0.f;                                            // unit rows: an accumulator column times 1/|query| is a cosine
        if (valid) {
            float q = 0.f;
            for (uint32_t j = 0; j < d4; ++j) {
                const float4 x = __ldg(row + j);
                q = fmaf(x.x, x.x, q); q = fmaf(x.y, x.y, q); q = fmaf(x.z, x.z, q); q = fmaf(x.w, x.w, q);
            }
            ic = q > 0.f ? 1.0f / sqrtf(q) : 0.f;
            inv_norm[c] = ic;
        }
        for (uint32_t kb = 0; kb < nkb; ++kb) {
            unsigned char *dst = out + (tile * nkb + kb) * (size_t)kBStage + r * 16;
#pragma unroll
            for (int ch = 0; ch < kScCh; ++ch) {
                const uint32_t c4 = kb * (kScKB / 4) + 2 * ch;
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
                if (valid && c4 < d4) x = __ldg(row + c4);
                if (valid && c4 + 1 < d4) y = __ldg(row + c4 + 1);
                *reinterpret_cast<uint4 *>(dst + ch * kBChunk) =
                    make_uint4(bf16x2(x.x * ic, x.y * ic), bf16x2(x.z * ic, x.w * ic), bf16x2(y.x * ic, y.y * ic), bf16x2(y.z * ic, y.w * ic));
            }
        }
    }
}

// fp32 dot product of two table rows by the whole warp (every lane gets the sum)
// The same packed copy for rows of at most 320 columns, staged through shared memory: sixteen warps read
// the tile's rows with coalesced 16-byte loads (four rows per warp in flight), reduce the norm with
// shuffles and write the scaled bf16 values into a shared-memory image of the tile (chunk stride padded
// by 16 bytes against bank conflicts); the image then goes out as one contiguous run.  Every row is read
// once and every output byte written once, in whole lines (the one-thread-per-row kernel above moves
// 1.5 times the bytes).
constexpr int kPackThreads = 512;
constexpr uint32_t kPackMaxF = 96;                                // float4 slots per row a lane can hold (3 x 32)
template <int NT>
__global__ void __launch_bounds__(kPackThreads)
topk_pack_candidates_smem_kernel(const float *__restrict__ table, float *__restrict__ inv_norm, uint32_t d4, uint32_t ld4,
                                 uint64_t cand_lo, uint64_t nc, uint64_t tiles, uint32_t nkb, unsigned char *__restrict__ out)
{
    extern __shared__ __align__(16) unsigned char pack_stage[];
    constexpr uint32_t kChunk = NT * 16, kPad = kChunk + 16;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t nf = nkb * (kScKB / 4);                         // float4 slots per row of the packed copy (zeros from d4 on)
    for (uint64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        for (uint32_t r0 = warp * 4; r0 < (uint32_t)NT; r0 += (kPackThreads / 32) * 4) {
            float4 x[4][3];
            bool valid[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const uint64_t c = tile * NT + r0 + t;
                valid[t] = c < nc;
                const float4 *row = reinterpret_cast<const float4 *>(table) + (size_t)(cand_lo + (valid[t] ? c : 0)) * ld4;
#pragma unroll
                for (int k = 0; k < 3; ++k) {
                    const uint32_t f = lane + 32u * k;
                    x[t][k] = valid[t] && f < d4 ? __ldg(row + f) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                float q = 0.f;
#pragma unroll
                for (int k = 0; k < 3; ++k) {
                    q = fmaf(x[t][k].x, x[t][k].x, q); q = fmaf(x[t][k].y, x[t][k].y, q);
                    q = fmaf(x[t][k].z, x[t][k].z, q); q = fmaf(x[t][k].w, x[t][k].w, q);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(kFullMask, q, o);
                const float ic = q > 0.f ? 1.0f / sqrtf(q) : 0.f;   // unit rows: an accumulator column times 1/|query| is a cosine
                if (lane == 0 && valid[t]) inv_norm[tile * NT + r0 + t] = ic;
#pragma unroll
                for (int k = 0; k < 3; ++k) {
                    const uint32_t f = lane + 32u * k;
                    if (f < nf)
                        *reinterpret_cast<uint2 *>(pack_stage + (size_t)(f >> 1) * kPad + (r0 + t) * 16u + (f & 1u) * 8u) =
                            make_uint2(bf16x2(x[t][k].x * ic, x[t][k].y * ic), bf16x2(x[t][k].z * ic, x[t][k].w * ic));
                }
            }
        }
        __syncthreads();
        uint4 *dst = reinterpret_cast<uint4 *>(out + tile * nkb * (size_t)(kScCh * kChunk));
        const uint32_t total = nkb * kScCh * NT;
        for (uint32_t i = threadIdx.x; i < total; i += kPackThreads)
            dst[i] = *reinterpret_cast<const uint4 *>(pack_stage + (size_t)(i / NT) * kPad + (i % NT) * 16u);
        __syncthreads();
    }
}

__device__ __forceinline__ float warp_row_dot(const float4 *__restrict__ T4, size_t a, size_t b, uint32_t d4, uint32_t ld4,
                                              uint32_t lane)
{
    float s = 0.f;
    for (uint32_t idx = lane; idx < d4; idx += 32) {
        const float4 x = __ldcg(T4 + a * ld4 + idx), y = __ldcg(T4 + b * ld4 + idx);
        s = fmaf(x.x, y.x, s); s = fmaf(x.y, y.y, s); s = fmaf(x.z, y.z, s); s = fmaf(x.w, y.w, s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFullMask, s, o);
    return s;
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0), "r"(0), "r"(0), "r"(0) : "memory");
}

// 32 consecutive fp32 columns of this thread's accumulator row (lane of tensor memory); asynchronous
// until tcgen05.wait::ld
__device__ __forceinline__ void tmem_ld32(uint32_t (&v)[32], uint32_t taddr)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr));
}

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Floats as unsigned integers in the same order (0 is below every float): for atomicMax.
__device__ __forceinline__ unsigned int ordered_bits(float f)
{
    const unsigned int u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ordered_float(unsigned int o)
{
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o);
}

// ================= epilogue of the screening kernels: one thread per query row =================
// Called by the four epilogue warps (threads 0..127) of a block whose accumulators (two buffers of
// 256 columns) start at tmem_base; `list` is the number of the partial list the block fills;
// arrive_tempty(b) tells the MMA issuer that this thread is done with accumulator buffer b.
template <typename Arrive>
__device__ __forceinline__ void screen_epilogue(const TcParams &p, const long long *qrow, uint64_t q0, uint64_t nc, uint64_t t_lo,
                                                uint64_t n_tiles, uint32_t tmem_base, uint64_t *tfull, volatile int *abort_flag,
                                                uint32_t list, Arrive &&arrive_tempty)
{
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t r = tid;
    const long long my_q = qrow[r];
    const bool live = q0 + r < p.m;
    const float4 *T4 = reinterpret_cast<const float4 *>(p.table);
    float *lc = p.part_cos + ((size_t)list * p.m + (q0 + r)) * p.K;      // this query's list (global, private)
    long long *li = p.part_ids + ((size_t)list * p.m + (q0 + r)) * p.K;
    float qinv = 0.f;
    if (my_q >= 0) {
        const float4 *row = T4 + (size_t)my_q * p.ld4;
        float s = 0.f;
        for (uint32_t j = 0; j < p.d4; ++j) {
            const float4 x = __ldcg(row + j);
            s = fmaf(x.x, x.x, s); s = fmaf(x.y, x.y, s); s = fmaf(x.z, x.z, s); s = fmaf(x.w, x.w, s);
        }
        qinv = s > 0.f ? 1.0f / sqrtf(s) : 0.f;
    }
    if (live) for (uint32_t s = 0; s < p.K; ++s) { lc[s] = 0.f; li[s] = -1; }
    const bool mine = my_q >= 0 && live;
    uint32_t have = 0;
    float thr = p.tau;
    // The blocks that work on other candidates of the same queries publish the K-th best cosine they
    // have reached (floor_q, raised by atomicMax); K candidates at or above it exist, so whatever is
    // below it cannot be among the query's final K, in any block.  Read once per tile.
    float flo = -INFINITY;
    // one chunk of 32 columns of the current tile (first candidate c0 + cc)
    uint64_t c0 = 0;
    auto screen_chunk = [&](const uint32_t (&v)[32], uint32_t cc) {
        __syncwarp();
        const float cut = fmaxf(have < p.K ? p.tau : fmaxf(p.tau, thr), flo) - kScreenEps;
        // the largest of the 32 columns, as a tree of three-input maxima (11 + 4 + 1 operations, depth 4)
        float t1[11];
#pragma unroll
        for (int j = 0; j < 10; ++j) t1[j] = max3(__uint_as_float(v[3 * j]), __uint_as_float(v[3 * j + 1]), __uint_as_float(v[3 * j + 2]));
        t1[10] = fmaxf(__uint_as_float(v[30]), __uint_as_float(v[31]));
        const float top = max3(max3(t1[0], t1[1], t1[2]), max3(t1[3], t1[4], t1[5]),
                               max3(max3(t1[6], t1[7], t1[8]), t1[9], t1[10]));
        const bool hit = mine && c0 + cc < nc && top * qinv >= cut;
        // a chunk with a column near the cut is rare: everything below sits behind one warp-wide branch
        if (!__any_sync(kFullMask, hit)) return;
        uint32_t maybe = 0u;
        if (hit) {                                                     // which of them?
#pragma unroll
            for (int j = 0; j < 32; ++j) maybe |= (__uint_as_float(v[j]) * qinv >= cut ? 1u : 0u) << j;
            const uint64_t left = nc - (c0 + cc);                      // candidates of the range from column cc on
            if (left < 32) maybe &= (1u << (uint32_t)left) - 1u;
        }
        // Exact pass: the set bits of all lanes, up to kExact queries (lanes) at a time.  The whole warp
        // works on each (query, candidate): 32 lanes on the fp32 dot product of the two table rows
        // (the loads of all kExact pairs are issued before the first sum is reduced), then on the
        // insertion into that query's sorted list, lane l holding entries l and l + 32.
        for (;;) {
            uint32_t owners = __ballot_sync(kFullMask, maybe != 0u);
            if (!owners) break;
            bool on[kExact];
            uint32_t src[kExact], hv[kExact];
            float th[kExact], fl[kExact], qi[kExact], dot[kExact], e0[kExact], e1[kExact], cinv[kExact];
            long long i0[kExact], i1[kExact], qr[kExact];
            uint64_t cnd[kExact];
#pragma unroll
            for (int e = 0; e < kExact; ++e) {
                on[e] = owners != 0u;
                src[e] = on[e] ? (uint32_t)__ffs((int)owners) - 1u : 0u;
                owners &= owners - 1u;
                const uint32_t j = __shfl_sync(kFullMask, (uint32_t)__ffs((int)maybe) - 1u, src[e]);
                cnd[e] = c0 + cc + j;
                qr[e] = qrow[warp * 32u + src[e]];
                hv[e] = __shfl_sync(kFullMask, have, src[e]);
                th[e] = __shfl_sync(kFullMask, thr, src[e]);
                fl[e] = __shfl_sync(kFullMask, flo, src[e]);
                qi[e] = __shfl_sync(kFullMask, qinv, src[e]);
                if (on[e] && lane == src[e]) maybe &= maybe - 1u;
                e0[e] = 0.f; e1[e] = 0.f; i0[e] = -1; i1[e] = -1; dot[e] = 0.f; cinv[e] = 0.f;
                if (on[e]) {
                    cinv[e] = __ldg(p.inv_norm + cnd[e]);                   // fetched with the rows, not after the sum
                    const size_t lb = ((size_t)list * p.m + (q0 + warp * 32u + src[e])) * p.K;
                    if (lane < hv[e]) { e0[e] = __ldcg(p.part_cos + lb + lane); i0[e] = __ldcg(p.part_ids + lb + lane); }
                    if (lane + 32u < hv[e]) { e1[e] = __ldcg(p.part_cos + lb + lane + 32u); i1[e] = __ldcg(p.part_ids + lb + lane + 32u); }
                }
            }
            for (uint32_t idx = lane; idx < p.d4; idx += 32) {
#pragma unroll
                for (int e = 0; e < kExact; ++e) {
                    if (on[e]) {
                        const float4 x = __ldcg(T4 + (size_t)qr[e] * p.ld4 + idx);
                        const float4 y = __ldcg(T4 + (size_t)(p.cand_lo + cnd[e]) * p.ld4 + idx);
                        dot[e] = fmaf(x.x, y.x, dot[e]); dot[e] = fmaf(x.y, y.y, dot[e]);
                        dot[e] = fmaf(x.z, y.z, dot[e]); dot[e] = fmaf(x.w, y.w, dot[e]);
                    }
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                for (int e = 0; e < kExact; ++e) dot[e] += __shfl_xor_sync(kFullMask, dot[e], o);
            }
#pragma unroll
            for (int e = 0; e < kExact; ++e) {
                if (!on[e]) continue;                                                   // same for every lane
                const float cs = dot[e] * qi[e] * cinv[e];
                const long long cid = (long long)(p.cand_lo + cnd[e]);
                if (!(cs > p.tau) || cid == qr[e] || (hv[e] == p.K && cs < th[e]) || cs < fl[e]) continue;
                const size_t lb = ((size_t)list * p.m + (q0 + warp * 32u + src[e])) * p.K;
                float *wl = p.part_cos + lb;
                long long *wi = p.part_ids + lb;
                const bool a0 = lane < hv[e] && !ranks_ahead_tc(cs, cid, e0[e], i0[e]);         // entries that stay ahead: a prefix
                const bool a1 = lane + 32u < hv[e] && !ranks_ahead_tc(cs, cid, e1[e], i1[e]);
                const uint32_t pos = (uint32_t)__popc(__ballot_sync(kFullMask, a0)) + (uint32_t)__popc(__ballot_sync(kFullMask, a1));
                const uint32_t km2 = p.K >= 2u ? p.K - 2u : 0u;
                const float e_km2 = km2 < 32u ? __shfl_sync(kFullMask, e0[e], km2) : __shfl_sync(kFullMask, e1[e], km2 - 32u);
                if (pos < p.K) {
                    if (lane < hv[e] && !a0 && lane + 1u < p.K) { wl[lane + 1u] = e0[e]; wi[lane + 1u] = i0[e]; }
                    if (lane + 32u < hv[e] && !a1 && lane + 33u < p.K) { wl[lane + 33u] = e1[e]; wi[lane + 33u] = i1[e]; }
                    if (lane == 0) { wl[pos] = cs; wi[pos] = cid; }
                    if (lane == src[e]) {
                        have = hv[e] < p.K ? hv[e] + 1u : p.K;
                        thr = have == p.K ? (pos == p.K - 1u ? cs : e_km2) : p.tau;
                        if (have == p.K) atomicMax(p.floor_q + (q0 + warp * 32u + src[e]), ordered_bits(thr));
                    }
                }
            }
            __syncwarp();
        }
    };
    for (uint64_t i = 0; i < n_tiles; ++i) {
        const uint32_t b = (uint32_t)(i & 1);
        c0 = (t_lo + i) * kTcN;
        if (mine) { const unsigned int o = __ldcg(p.floor_q + (q0 + r)); if (o) flo = ordered_float(o); }
        // the tensor-memory loads below are warp-wide: the whole warp goes on or gives up together
        if (!__all_sync(kFullMask, mbar_wait(tfull + b, (uint32_t)((i >> 1) & 1), abort_flag))) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // Two chunks of 32 accumulator columns are in flight: the load of chunk k + 1 is issued before
        // chunk k is looked at.  The candidate rows were packed as unit vectors, so a column times
        // 1/|query| is the screened cosine; the largest of the 32 decides whether the chunk needs a
        // closer look at all.
        uint32_t va[32], vb[32];
        tmem_ld32(va, tmem_base + ((warp * 32u) << 16) + b * kTcN);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll 1
        for (uint32_t cc = 0; cc < (uint32_t)kTcN; cc += 64) {
            tmem_ld32(vb, tmem_base + ((warp * 32u) << 16) + b * kTcN + cc + 32u);
            screen_chunk(va, cc);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (cc + 64u < (uint32_t)kTcN) tmem_ld32(va, tmem_base + ((warp * 32u) << 16) + b * kTcN + cc + 64u);
            screen_chunk(vb, cc + 32u);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        arrive_tempty(b);                                     // this accumulator buffer may be overwritten
    }
}

// RES: the query block is resident in shared memory (d <= 320); otherwise its K-blocks stream through
// the stages beside the candidates' (8 KB + 16 KB per stage).
template <bool RES>
__global__ void __launch_bounds__(kScThreads, 1)
topk_cosine_screen_kernel(TcParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    // RES: [kScMaxKB query K-blocks][kScStages candidate stages]; else [kScStages stages of (kScKPS query K-blocks, kScKPS candidate K-blocks)]
    constexpr int kStage = kScKPS * (RES ? kScStageBytes : kScABlock + kScStageBytes);
    unsigned char *a_op = smem;
    unsigned char *b_op = smem + (RES ? kScMaxKB * kScABlock : kScKPS * kScABlock);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + (RES ? kScMaxKB * kScABlock : 0) + kScStages * kStage);
    uint64_t *empty = full + kScStages;
    uint64_t *tfull = empty + kScStages;
    uint64_t *tempty = tfull + 2;
    uint64_t *afull = tempty + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(afull + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    long long *qrow = reinterpret_cast<long long *>(tmem_slot + 2);          // [128]

    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint64_t q0 = (uint64_t)blockIdx.x * kTcM;
    const uint64_t nc = p.cand_hi - p.cand_lo;
    const uint64_t tiles = (nc + kTcN - 1) / kTcN;
    const uint64_t t_lo = tiles * blockIdx.y / p.splits, t_hi = tiles * (blockIdx.y + 1) / p.splits;
    const uint32_t nkb = (4u * p.d4 + kScKB - 1) / kScKB;
    const uint64_t n_tiles = t_hi - t_lo;

    if (tid == 0) {
        for (int s = 0; s < kScStages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull + b, 1); mbar_init(tempty + b, kTcM); }
        mbar_init(afull, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < (uint32_t)kTcM) {
        long long r = q0 + tid < p.m ? p.queries[q0 + tid] : -1;
        if (r < 0 || (unsigned long long)r >= p.vocab) r = -1;
        qrow[tid] = r;
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)), "r"(2 * kTcN));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4) {
        screen_epilogue(p, qrow, q0, nc, t_lo, n_tiles, tmem_base, tfull, abort_flag, blockIdx.y,
                        [&](uint32_t b) { mbar_arrive(tempty + b); });
    } else if (warp == 4) {
        // ================= MMA issue: one lane =================
        if (lane == 0) {
            // bf16 x bf16 -> fp32, both operands K-major, N = 256, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTcN >> 3) << 17) | ((uint32_t)(kTcM >> 4) << 24);
            bool ok = true;
            if (RES) {
                // the query block: one bulk copy per K-block, all on one barrier
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                             ::"r"(smem_addr(afull)), "r"(nkb * (uint32_t)kScABlock) : "memory");
                for (uint32_t kb = 0; kb < nkb; ++kb)
                    bulk_to_smem(a_op + (size_t)kb * kScABlock, p.qsplit + ((size_t)blockIdx.x * nkb + kb) * kScABlock,
                                 (uint32_t)kScABlock, afull);
                ok = mbar_wait(afull, 0u, abort_flag);
            }
            // One lane issues everything, so what it executes per MMA is what bounds the block when the
            // copies keep up: the descriptors of a tile's MMAs differ only in their address fields, which
            // advance by a constant per k-step (the K-blocks of an operand lie side by side), so the loop
            // body is two additions and the MMA.
            const uint32_t n16 = (4u * p.d4 + 15u) / 16u;                  // MMAs (K = 16) per tile; k-steps of pure padding are skipped
            constexpr uint32_t kPerStage = 2u * kScKPS;                     // MMAs per full stage
            constexpr uint64_t kAStep = (2u * kScAChunk) >> 4, kBStep = (2u * kScBChunk) >> 4, kStageStep = (uint32_t)kStage >> 4;
            const uint64_t adesc0 = umma_desc(smem_addr(a_op), kScAChunk, 128), bdesc0 = umma_desc(smem_addr(b_op), kScBChunk, 128);
            uint32_t s = 0, ph = 0;
            for (uint64_t i = 0; i < n_tiles && ok; ++i) {
                const uint32_t b = (uint32_t)(i & 1);
                ok = mbar_wait(tempty + b, (uint32_t)(((i >> 1) & 1) ^ 1), abort_flag);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t dst = tmem_base + b * kTcN;
                uint64_t qa = adesc0;
                uint32_t left = n16, acc = 0u;
                while (left && ok) {
                    ok = mbar_wait(full + s, ph, abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    uint64_t cb = bdesc0 + s * kStageStep;
                    if (!RES) qa = adesc0 + s * kStageStep;
                    const uint32_t n = left < kPerStage ? left : kPerStage;
                    for (uint32_t t = 0; t < n; ++t, qa += kAStep, cb += kBStep, acc = 1u) umma_bf16(dst, qa, cb, idesc, acc);
                    left -= n;
                    umma_commit(empty + s);                       // the stage is free once these MMAs have read it
                    if (++s == (uint32_t)kScStages) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(tfull + b);                   // the tile's accumulator is complete
            }
        }
    } else {
        // ================= producer: one lane =================
        // one bulk copy per stage, issued when the MMAs that read the stage's previous contents have
        // committed; its bytes complete the stage's "full" barrier
        if (lane == 0) {
            uint64_t g = 0;                                                   // stages issued so far
            uint32_t s = 0, ph = 1u;
            const unsigned char *tile = p.ctiles + t_lo * nkb * (size_t)kScStageBytes;
            const unsigned char *qsrc = RES ? nullptr : p.qsplit + (size_t)blockIdx.x * nkb * kScABlock;
            for (uint64_t i = 0; i < n_tiles; ++i, tile += (size_t)nkb * kScStageBytes) {
                uint32_t kb0 = 0;
                for (; kb0 < nkb; kb0 += kScKPS, ++g) {
                    if (!mbar_wait(empty + s, ph, abort_flag)) break;
                    const uint32_t nkbs = nkb - kb0 < (uint32_t)kScKPS ? nkb - kb0 : (uint32_t)kScKPS;  // K-blocks the stage holds
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                                 ::"r"(smem_addr(full + s)), "r"(nkbs * (uint32_t)(RES ? kScStageBytes : kScABlock + kScStageBytes)) : "memory");
                    if (!RES) bulk_to_smem(a_op + (size_t)s * kStage, qsrc + (size_t)kb0 * kScABlock, nkbs * (uint32_t)kScABlock, full + s);
                    bulk_to_smem(b_op + (size_t)s * kStage, tile + (size_t)kb0 * kScStageBytes, nkbs * (uint32_t)kScStageBytes, full + s);
                    if (++s == (uint32_t)kScStages) { s = 0; ph ^= 1u; }
                }
                if (kb0 < nkb) break;                                         // a wait ran out
            }
            if (*abort_flag) {
                // the block is giving up: let the copies still in flight land before shared memory is released
                for (uint64_t j = g > (uint64_t)kScStages ? g - kScStages : 0; j < g; ++j)
                    for (uint32_t spin = 0; spin < kTcSpinLimit; ++spin)
                        if (mbar_try(full + j % kScStages, (uint32_t)((j / kScStages) & 1))) break;
            }
        }
    }
    // ================= common exit =================
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0 && *abort_flag) atomicExch(p.error, 1);
    if (warp == 4) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kTcN));
    }
}

// =================================================================================================
// The screening kernel on a pair of SMs (`cta_group::2`): a cluster of two thread blocks, each with
// its own resident query block (M = 2 x 128 accumulator rows) and HALF of every candidate tile (N = 256
// as 2 x 128 rows), so every candidate byte that an SM pulls through L2 now serves 256 queries and the
// stage memory of both SMs works for one tile stream.  The even block of the pair (the leader) issues
// the MMAs for both; each block's tensor core reads its own query block and both halves of the tile and
// writes the 128 x 256 accumulator of its own queries into its own tensor memory, where the block's
// epilogue warps screen it exactly as in the one-block kernel.
//
// Hand-overs (every barrier lives in one block's shared memory; nothing is broadcast):
//   full[s]   own half of stage s has landed (bulk copy, complete_tx)          waited by: leader's MMA lane / follower's relay
//   fullF[s]  (leader) the follower's half has landed; its relay lane arrives remotely
//   empty[s]  the MMAs that read stage s are done: leader's by tcgen05.commit, follower's by a remote
//             arrival from the leader's relay lane, which waits on the leader's empty[s]
//   tfull[b]  accumulator b complete: leader's by tcgen05.commit, follower's through the leader's second relay lane
//   tempty[b] (leader) all 256 epilogue threads of the pair are done with accumulator b (128 remote arrivals)
// All waits are the time-limited mbar_wait; a block that gives up still reaches the cluster barrier at
// the end, so its partner (whose waits then run out too) is never left behind.
constexpr int kPrStages = 3;
constexpr int kPrKPS = 5;                                         // K-blocks per stage
constexpr int kPrHalf = kTcN / 2;                                 // candidate rows of a tile per block
constexpr int kPrBChunk = kPrHalf * 16;
constexpr int kPrKBlock = kScCh * kPrBChunk;                      // one K-block of a half tile: 8 KB
constexpr int kPrStage = kPrKPS * kPrKBlock;                      // 40 KB
constexpr int kPrThreads = 8 * 32;                                // 4 epilogue warps, MMA, producer, two relay warps

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrival on the barrier at the same shared-memory offset in block `rank` of the cluster
__device__ __forceinline__ void mbar_arrive_in(uint64_t *bar, uint32_t rank)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_addr(bar)), "r"(rank));
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
// the time-limited wait for a barrier that another block of the cluster arrives at
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    unsigned long long t0 = 0;
    for (uint32_t spin = 0; spin < (1u << 30); ++spin) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(smem_addr(bar)), "r"(parity) : "memory");
        if (done) return true;
        if ((spin & 1023u) == 1023u) {
            if (*abort_flag) return false;
            if (!t0) t0 = global_ns();
            else if (global_ns() - t0 > kTcWaitNs) break;
        }
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0) : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPrThreads, 1)
topk_cosine_screen_pair_kernel(TcParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *a_op = smem;                                              // [kScMaxKB] K-blocks of the own query block
    unsigned char *b_op = smem + kScMaxKB * kScABlock;                       // [kPrStages] stages of the own half tile
    uint64_t *full = reinterpret_cast<uint64_t *>(b_op + kPrStages * kPrStage);
    uint64_t *fullF = full + kPrStages;
    uint64_t *empty = fullF + kPrStages;
    uint64_t *tfull = empty + kPrStages;
    uint64_t *tempty = tfull + 2;
    uint64_t *afull = tempty + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(afull + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    long long *qrow = reinterpret_cast<long long *>(tmem_slot + 2);          // [128]

    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_rank();                                     // 0: leader, 1: follower
    const bool leader = rank == 0;
    const uint64_t q0 = (uint64_t)blockIdx.x * kTcM;
    const uint64_t nc = p.cand_hi - p.cand_lo;
    const uint64_t tiles = (nc + kTcN - 1) / kTcN;                            // tiles of 256 candidates, as two half tiles in the packed copy
    const uint64_t t_lo = tiles * blockIdx.y / p.splits, t_hi = tiles * (blockIdx.y + 1) / p.splits;
    const uint32_t nkb = (4u * p.d4 + kScKB - 1) / kScKB;
    const uint32_t nst = (nkb + kPrKPS - 1) / kPrKPS;
    const uint64_t n_tiles = t_hi - t_lo;
    const uint64_t total_g = n_tiles * nst;

    if (tid == 0) {
        for (int s = 0; s < kPrStages; ++s) { mbar_init(full + s, 1); mbar_init(fullF + s, 1); mbar_init(empty + s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull + b, 1); mbar_init(tempty + b, 2 * kTcM); }
        mbar_init(afull, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < (uint32_t)kTcM) {
        long long r = q0 + tid < p.m ? p.queries[q0 + tid] : -1;
        if (r < 0 || (unsigned long long)r >= p.vocab) r = -1;
        qrow[tid] = r;
    }
    if (warp == 4) {       // the same warp of both blocks, the same slot: the pair's tensor memory is allocated together
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)), "r"(2 * kTcN));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync_all();                                                       // both blocks' barriers exist before anyone arrives remotely
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4) {
        if (leader)
            screen_epilogue(p, qrow, q0, nc, t_lo, n_tiles, tmem_base, tfull, abort_flag, blockIdx.y,
                            [&](uint32_t b) { mbar_arrive(tempty + b); });
        else
            screen_epilogue(p, qrow, q0, nc, t_lo, n_tiles, tmem_base, tfull, abort_flag, blockIdx.y,
                            [&](uint32_t b) { mbar_arrive_in(tempty + b, 0u); });
    } else if (warp == 4) {
        if (lane == 0) {
            // the own query block: one bulk copy per K-block, all on one barrier
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         ::"r"(smem_addr(afull)), "r"(nkb * (uint32_t)kScABlock) : "memory");
            for (uint32_t kb = 0; kb < nkb; ++kb)
                bulk_to_smem(a_op + (size_t)kb * kScABlock, p.qsplit + ((size_t)blockIdx.x * nkb + kb) * kScABlock,
                             (uint32_t)kScABlock, afull);
            bool ok = mbar_wait(afull, 0u, abort_flag);
            if (leader) {
                // bf16 x bf16 -> fp32, both operands K-major, M = 256 and N = 256 over the pair
                const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTcN >> 3) << 17) | ((uint32_t)((2 * kTcM) >> 4) << 24);
                // as in the one-block kernel: address fields advance by a constant per k-step
                const uint32_t n16 = (4u * p.d4 + 15u) / 16u;
                constexpr uint32_t kPerStage = 2u * kPrKPS;
                constexpr uint64_t kAStep = (2u * kScAChunk) >> 4, kBStep = (2u * kPrBChunk) >> 4, kStageStep = (uint32_t)kPrStage >> 4;
                const uint64_t adesc0 = umma_desc(smem_addr(a_op), kScAChunk, 128), bdesc0 = umma_desc(smem_addr(b_op), kPrBChunk, 128);
                uint32_t s = 0, ph = 0;
                for (uint64_t i = 0; i < n_tiles && ok; ++i) {
                    const uint32_t b = (uint32_t)(i & 1);
                    ok = mbar_wait_cluster(tempty + b, (uint32_t)(((i >> 1) & 1) ^ 1), abort_flag);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t dst = tmem_base + b * kTcN;
                    uint64_t qa = adesc0;
                    uint32_t left = n16, acc = 0u;
                    while (left && ok) {
                        ok = mbar_wait(full + s, ph, abort_flag) && mbar_wait_cluster(fullF + s, ph, abort_flag);
                        if (!ok) break;
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        uint64_t cb = bdesc0 + s * kStageStep;
                        const uint32_t n = left < kPerStage ? left : kPerStage;
                        for (uint32_t t = 0; t < n; ++t, qa += kAStep, cb += kBStep, acc = 1u) umma_bf16_pair(dst, qa, cb, idesc, acc);
                        left -= n;
                        umma_commit_pair(empty + s);
                        if (++s == (uint32_t)kPrStages) { s = 0; ph ^= 1u; }
                    }
                    if (ok) umma_commit_pair(tfull + b);
                }
            }
        }
    } else if (warp == 5) {
        // producer: the own half of every stage
        if (lane == 0) {
            uint64_t g = 0;                                                   // stages issued so far
            uint32_t s = 0, ph = 1u;
            // half tile number 2 T + rank of the packed copy (tiles of 128 rows)
            const unsigned char *tile = p.ctiles + (2 * t_lo + rank) * nkb * (size_t)kPrKBlock;
            for (uint64_t i = 0; i < n_tiles; ++i, tile += 2 * (size_t)nkb * kPrKBlock) {
                uint32_t kb0 = 0;
                for (; kb0 < nkb; kb0 += kPrKPS, ++g) {
                    if (!(leader ? mbar_wait(empty + s, ph, abort_flag) : mbar_wait_cluster(empty + s, ph, abort_flag))) break;
                    const uint32_t nkbs = nkb - kb0 < (uint32_t)kPrKPS ? nkb - kb0 : (uint32_t)kPrKPS;
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                                 ::"r"(smem_addr(full + s)), "r"(nkbs * (uint32_t)kPrKBlock) : "memory");
                    bulk_to_smem(b_op + (size_t)s * kPrStage, tile + (size_t)kb0 * kPrKBlock, nkbs * (uint32_t)kPrKBlock, full + s);
                    if (++s == (uint32_t)kPrStages) { s = 0; ph ^= 1u; }
                }
                if (kb0 < nkb) break;                                         // a wait ran out
            }
            if (*abort_flag) {
                for (uint64_t j = g > (uint64_t)kPrStages ? g - kPrStages : 0; j < g; ++j)
                    for (uint32_t spin = 0; spin < kTcSpinLimit; ++spin)
                        if (mbar_try(full + j % kPrStages, (uint32_t)((j / kPrStages) & 1))) break;
            }
        }
    } else if (warp == 6) {
        if (lane == 0) {
            if (leader) {
                // relay: a stage whose MMAs are done is free in the follower as well
                for (uint64_t g = 0; g < total_g; ++g) {
                    const uint32_t s = (uint32_t)(g % kPrStages);
                    if (!mbar_wait(empty + s, (uint32_t)((g / kPrStages) & 1), abort_flag)) break;
                    mbar_arrive_in(empty + s, 1u);
                }
            } else {
                // relay: the follower's half of a stage (and, first of all, its query block) has landed
                bool ok = mbar_wait(afull, 0u, abort_flag);
                for (uint64_t g = 0; g < total_g && ok; ++g) {
                    const uint32_t s = (uint32_t)(g % kPrStages);
                    ok = mbar_wait(full + s, (uint32_t)((g / kPrStages) & 1), abort_flag);
                    if (ok) mbar_arrive_in(fullF + s, 0u);
                }
            }
        }
    } else {
        if (lane == 0 && leader) {
            // relay: a complete accumulator is complete in the follower's tensor memory as well
            for (uint64_t i = 0; i < n_tiles; ++i) {
                const uint32_t b = (uint32_t)(i & 1);
                if (!mbar_wait(tfull + b, (uint32_t)((i >> 1) & 1), abort_flag)) break;
                mbar_arrive_in(tfull + b, 1u);
            }
        }
    }
    // ================= common exit =================
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0 && *abort_flag) atomicExch(p.error, 1);
    cluster_sync_all();                                   // neither block leaves while its partner may still reach into it
    if (warp == 4) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kTcN));
    }
}

static size_t topk_screen_pair_smem_bytes()
{
    return (size_t)kScMaxKB * kScABlock + (size_t)kPrStages * kPrStage + (3 * kPrStages + 5) * 8 + 8 + kTcM * 8 + 128;
}

// The give-up path of the retrieval kernels on its own: one block waits, with the kernels' own wait
// routine and a short limit, on a barrier that nobody arrives at; when the limit has passed it raises
// the error word exactly as a retrieval block does, and returns.
__global__ void __launch_bounds__(64)
bounded_wait_selftest_kernel(unsigned long long limit_ns, int *error)
{
    __shared__ uint64_t bar;
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // lane 0 of warp 0 waits for the arrival that never comes; lane 0 of warp 1 waits behind it and must
    // leave through the abort flag as soon as the first has given up
    if ((threadIdx.x & 31) == 0) mbar_wait(&bar, 0u, abort_flag, threadIdx.x == 0 ? limit_ns : 100 * limit_ns);
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicExch(error, 1);
}

int launch_bounded_wait_selftest(uint32_t timeout_ms, int *error, cudaStream_t s)
{
    bounded_wait_selftest_kernel<<<1, 64, 0, s>>>((unsigned long long)timeout_ms * 1000000ull, error);
    return cudaGetLastError() != cudaSuccess ? -1 : 1;
}

static size_t topk_screen_smem_bytes(bool resident)
{
    const size_t operands = resident ? (size_t)kScMaxKB * kScABlock + (size_t)kScStages * kScKPS * kScStageBytes
                                     : (size_t)kScStages * kScKPS * (kScABlock + kScStageBytes);
    return operands + (2 * kScStages + 5) * 8 + 8 + kTcM * 8 + 128;
}

// whether the query block of rows of d columns can stay in shared memory
static bool topk_screen_resident(uint32_t d) { return (d + kScKB - 1) / kScKB <= (uint32_t)kScMaxKB; }

size_t topk_tc_smem_bytes()
{
    return (size_t)kTcStages * kTcStageBytes + (2 * kTcStages + 4) * 8 + 16 + kTcM * 8 + 8 * kTcN * 4 + 128;
}

size_t topk_tc_qsplit_bytes(uint64_t m, uint32_t d)
{
    const uint64_t qblocks = (m + kTcM - 1) / kTcM, nkb = (d + kTcKB - 1) / kTcKB;
    return (size_t)(qblocks * nkb * 2 * kTcOperand);          // the screening layout needs less (kScABlock per K-block)
}

// Screening kernel: candidates are handled in chunks of at most kScChunk rows and at most kScScratch
// bytes of packed bf16 copy (the scratch `ctiles`); every chunk has its own `splits` partial lists.
constexpr uint64_t kScChunk = 1ull << 22;
constexpr uint64_t kScScratch = 2752512000ull;                  // 2^22 rows of 320 columns, plus a little

uint64_t topk_screen_chunk(uint64_t nc, uint32_t d)
{
    const uint64_t nkb = (d + kScKB - 1) / kScKB;
    uint64_t chunk = kScScratch / (nkb * kScStageBytes) * kTcN;     // whole tiles
    if (chunk > kScChunk) chunk = kScChunk;
    if (chunk < (uint64_t)kTcN) chunk = kTcN;
    return nc < chunk ? nc : chunk;
}

size_t topk_screen_ctiles_bytes(uint64_t nc, uint32_t d)
{
    const uint64_t chunk = topk_screen_chunk(nc, d), tiles = (chunk + kTcN - 1) / kTcN, nkb = (d + kScKB - 1) / kScKB;
    return (size_t)(tiles * nkb * kScStageBytes);
}

// Returns the launches made, or -1 on a launch error.  Results go to part_* ([lists][m][K], lists = splits, or
// chunks x splits for the screening kernel); the caller merges.
int launch_topk_tc(const float *table, uint32_t d, uint32_t ld, uint64_t vocab, const long long *queries, uint64_t m,
                   uint64_t cand_lo, uint64_t cand_hi, uint32_t K, float tau, float *inv_norm,
                   unsigned char *qsplit, unsigned char *ctiles, unsigned int *floor_q, float *part_cos, long long *part_ids,
                   uint32_t splits, int *error, bool screen, bool pairs, int sms, cudaStream_t s)
{
    if (m == 0) return 0;
    const unsigned qblocks = (unsigned)((m + kTcM - 1) / kTcM);
    TcParams p;
    p.qsplit = qsplit; p.ctiles = ctiles; p.floor_q = floor_q;
    p.table = table; p.queries = queries; p.inv_norm = inv_norm; p.part_cos = part_cos; p.part_ids = part_ids;
    p.error = error; p.m = m; p.vocab = vocab; p.cand_lo = cand_lo; p.cand_hi = cand_hi;
    p.d4 = d / 4; p.ld4 = ld / 4; p.K = K; p.splits = splits; p.tau = tau;
    dim3 grid(qblocks, splits);
    if (!screen) {
        const uint32_t nkb = (d + kTcKB - 1) / kTcKB;
        topk_split_queries_kernel<<<qblocks * nkb, 256, 0, s>>>(table, queries, m, vocab, d / 4, ld / 4, nkb, qsplit);
        if (cudaGetLastError() != cudaSuccess) return -1;
        const size_t sm = topk_tc_smem_bytes();
        if (cudaFuncSetAttribute(topk_cosine_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess)
            return -1;
        topk_cosine_tc_kernel<<<grid, kTcThreads, sm, s>>>(p);
        if (cudaGetLastError() != cudaSuccess) return -1;
        return 2;
    }
    const uint32_t nkb = (d + kScKB - 1) / kScKB;
    topk_round_queries_kernel<<<((qblocks + 1) / 2 * 2) * nkb, 256, 0, s>>>(table, queries, m, vocab, d / 4, ld / 4, nkb, qsplit);
    if (cudaGetLastError() != cudaSuccess) return -1;
    if (cudaMemsetAsync(floor_q, 0, m * sizeof(unsigned int), s) != cudaSuccess) return -1;   // 0 = no floor yet
    const bool resident = topk_screen_resident(d);
    // on request, with more than one query block of resident width: pairs of blocks on pairs of SMs share every candidate tile
    const bool pair = pairs && resident && qblocks >= 2;
    const size_t sm = pair ? topk_screen_pair_smem_bytes() : topk_screen_smem_bytes(resident);
    const void *kernel = pair ? (const void *)topk_cosine_screen_pair_kernel
                         : resident ? (const void *)topk_cosine_screen_kernel<true> : (const void *)topk_cosine_screen_kernel<false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess) return -1;
    if (pair) grid.x = (qblocks + 1) / 2 * 2;                  // whole pairs; the rows of a padded block are zeros
    int launched = 1;
    const uint64_t nc = cand_hi - cand_lo, chunk = topk_screen_chunk(nc, d);
    uint64_t list = 0;
    for (uint64_t c0 = 0; c0 < nc; c0 += chunk, ++list) {
        const uint64_t n = nc - c0 < chunk ? nc - c0 : chunk;
        const uint64_t tiles = (n + kTcN - 1) / kTcN;
        if (nkb * (kScKB / 4) <= kPackMaxF && nkb <= (uint32_t)kScMaxKB) {               // rows of at most 320 columns: through shared memory
            const size_t psm = (size_t)nkb * kScCh * ((pair ? kPrHalf : kTcN) * 16 + 16);
            const void *pk = pair ? (const void *)topk_pack_candidates_smem_kernel<kPrHalf> : (const void *)topk_pack_candidates_smem_kernel<kTcN>;
            if (cudaFuncSetAttribute(pk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)psm) != cudaSuccess) return -1;
            if (pair)
                topk_pack_candidates_smem_kernel<kPrHalf><<<sms * 2, kPackThreads, psm, s>>>(table, inv_norm + c0, d / 4, ld / 4, cand_lo + c0, n, 2 * tiles, nkb, ctiles);
            else
                topk_pack_candidates_smem_kernel<kTcN><<<sms, kPackThreads, psm, s>>>(table, inv_norm + c0, d / 4, ld / 4, cand_lo + c0, n, tiles, nkb, ctiles);
        } else if (pair)
            topk_pack_candidates_kernel<kPrHalf><<<sms * 32, kPrHalf, 0, s>>>(table, inv_norm + c0, d / 4, ld / 4, cand_lo + c0, n, 2 * tiles, nkb, ctiles);
        else
            topk_pack_candidates_kernel<kTcN><<<sms * 16, kTcN, 0, s>>>(table, inv_norm + c0, d / 4, ld / 4, cand_lo + c0, n, tiles, nkb, ctiles);
        if (cudaGetLastError() != cudaSuccess) return -1;
        p.cand_lo = cand_lo + c0; p.cand_hi = cand_lo + c0 + n;
        p.inv_norm = inv_norm + c0;
        p.part_cos = part_cos + list * splits * m * K;
        p.part_ids = part_ids + list * splits * m * K;
        if (pair) topk_cosine_screen_pair_kernel<<<grid, kPrThreads, sm, s>>>(p);
        else if (resident) topk_cosine_screen_kernel<true><<<grid, kScThreads, sm, s>>>(p);
        else topk_cosine_screen_kernel<false><<<grid, kScThreads, sm, s>>>(p);
        if (cudaGetLastError() != cudaSuccess) return -1;
        launched += 2;
    }
    return launched;
}

}  // namespace w2v

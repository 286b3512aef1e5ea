// Cosine retrieval on the tensor cores (tcgen05, TMEM accumulators), same contract as the fp32
// kernel in w2v_topk.cu.
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
// has an iteration limit, after which the block raises the error flag and leaves through the common
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
// another thread has already given up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    for (uint32_t spin = 0; spin < kTcSpinLimit; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 1023u) == 1023u && *abort_flag) return false;
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
// Screening variant.  One TF32 MMA per product instead of three: the accumulator then holds the dot
// product to about 1e-3 of |a||b| only (the query side is rounded to TF32 by a pre-pass, the
// candidate side is read by the tensor core as it lies in memory, i.e. truncated: relative errors
// of at most 2^-11 and 2^-10 per factor, so by Cauchy-Schwarz the cosine is off by less than
// 2^-11 + 2^-10 + 2^-20 = 1.47e-3; the fp32 accumulation adds some 1e-5).  That is enough to
// decide that a candidate cannot reach a query's current cut.  Only a candidate whose approximate
// cosine comes within kScreenEps of the cut is looked at again: its warp computes the fp32 dot
// product of the two rows from the table, and that exact cosine goes to the sorted list.  With a
// list of K the number of such candidates is about K ln(n / K) per query, against n screened.
//
// The query block stays in shared memory for the whole kernel (d <= 320: 160 KB), so only candidate
// rows stream: 128 query rows x 256 candidates per tile, two 32-column stages of candidates.
constexpr float kScreenEps = 2e-3f;
constexpr int kScMaxKB = 10;                                     // K-blocks of 32 columns that fit: d <= 320
constexpr int kScAChunk = kTcM * 16;                             // query operand: no padding (filled by bulk copies)
constexpr int kScABlock = 8 * kScAChunk;                         // bytes of one K-block of the query operand
constexpr int kScStageBytes = kTcOperandC;                       // one stage = one candidate operand block
constexpr int kScGroups = 3;                                     // loader groups: 96 KB of candidate rows in flight in registers
constexpr int kScThreads = 5 * 32 + kScGroups * kTcLoaders;

// Query rows of one block, rounded to TF32, in the layout of the shared-memory operand
// ([K-block][16-byte chunk][row][16 B]).  One block per (query block, K-block).
__global__ void __launch_bounds__(256)
topk_round_queries_kernel(const float *__restrict__ table, const long long *__restrict__ queries, uint64_t m,
                          uint64_t vocab, uint32_t d4, uint32_t ld4, uint32_t nkb, unsigned char *__restrict__ qtf32)
{
    const uint32_t qb = blockIdx.x / nkb, kb = blockIdx.x % nkb;
    unsigned char *dst = qtf32 + ((size_t)qb * nkb + kb) * kScABlock;
    const float4 *T4 = reinterpret_cast<const float4 *>(table);
    for (uint32_t e = threadIdx.x; e < (uint32_t)kTcM * 8; e += blockDim.x) {
        const uint32_t r = e >> 3, ch = e & 7;
        const uint64_t qi = (uint64_t)qb * kTcM + r;
        long long row = qi < m ? queries[qi] : -1;
        if (row < 0 || (unsigned long long)row >= vocab) row = -1;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row >= 0 && kb * 8 + ch < d4) x = __ldcg(T4 + (size_t)row * ld4 + (kb * 8 + ch));
        *reinterpret_cast<float4 *>(dst + ch * kScAChunk + r * 16) =
            make_float4(tf32_round(x.x), tf32_round(x.y), tf32_round(x.z), tf32_round(x.w));
    }
}

// fp32 dot product of two table rows by the whole warp (every lane gets the sum)
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

__global__ void __launch_bounds__(kScThreads, 1)
topk_cosine_screen_kernel(TcParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *a_op = smem;                                              // [kScMaxKB] query K-blocks
    unsigned char *b_op = smem + kScMaxKB * kScABlock;                       // [kTcStages] candidate stages
    uint64_t *full = reinterpret_cast<uint64_t *>(b_op + kTcStages * kScStageBytes);
    uint64_t *empty = full + kTcStages;
    uint64_t *tfull = empty + kTcStages;
    uint64_t *tempty = tfull + 2;
    uint64_t *afull = tempty + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(afull + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    volatile uint32_t *consumed = reinterpret_cast<volatile uint32_t *>(tmem_slot + 2);   // [kTcStages] uses of a stage the MMAs are done with
    long long *qrow = reinterpret_cast<long long *>(tmem_slot + 4);          // [128]

    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint64_t q0 = (uint64_t)blockIdx.x * kTcM;
    const uint64_t nc = p.cand_hi - p.cand_lo;
    const uint64_t tiles = (nc + kTcN - 1) / kTcN;
    const uint64_t t_lo = tiles * blockIdx.y / p.splits, t_hi = tiles * (blockIdx.y + 1) / p.splits;
    const uint32_t nkb = (4u * p.d4 + kTcKB - 1) / kTcKB;
    const uint64_t n_tiles = t_hi - t_lo;

    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) { mbar_init(full + s, kTcLoaders); mbar_init(empty + s, 1); consumed[s] = 0u; }
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
        // ================= epilogue: one thread per query row =================
        const uint32_t r = tid;
        const long long my_q = qrow[r];
        const bool live = q0 + r < p.m;
        const float4 *T4 = reinterpret_cast<const float4 *>(p.table);
        float *lc = p.part_cos + ((size_t)blockIdx.y * p.m + (q0 + r)) * p.K;      // this query's list (global, private)
        long long *li = p.part_ids + ((size_t)blockIdx.y * p.m + (q0 + r)) * p.K;
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
        for (uint64_t i = 0; i < n_tiles; ++i) {
            const uint32_t b = (uint32_t)(i & 1);
            const uint64_t c0 = (t_lo + i) * kTcN;
            // the tensor-memory loads below are warp-wide: the whole warp goes on or gives up together
            if (!__all_sync(kFullMask, mbar_wait(tfull + b, (uint32_t)((i >> 1) & 1), abort_flag))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
            for (uint32_t cc = 0; cc < (uint32_t)kTcN; cc += 32) {
                uint32_t v[32];
                __syncwarp();
                // lane l: 1/|x| of candidate cc + l of the tile (0 past the end of the range)
                const float icv = c0 + cc + lane < nc ? __ldg(p.inv_norm + c0 + cc + lane) : 0.f;
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
                // screen: bit j = candidate cc + j may reach this query's cut
                const float cut = (have < p.K ? p.tau : fmaxf(p.tau, thr)) - kScreenEps;
                uint32_t maybe = 0u;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float ic = __shfl_sync(kFullMask, icv, j);
                    maybe |= (__uint_as_float(v[j]) * qinv * ic >= cut ? 1u : 0u) << j;
                }
                const uint64_t left = nc - (c0 + cc);                  // candidates of the range from column cc on
                if (!mine || c0 + cc >= nc) maybe = 0u;
                else if (left < 32) maybe &= (1u << (uint32_t)left) - 1u;
                // exact pass, one (query, candidate) at a time, the whole warp on one dot product
                for (;;) {
                    const uint32_t owners = __ballot_sync(kFullMask, maybe != 0u);
                    if (!owners) break;
                    const uint32_t src = (uint32_t)__ffs((int)owners) - 1u;
                    const uint32_t j = __shfl_sync(kFullMask, (uint32_t)__ffs((int)maybe) - 1u, src);
                    const long long qr = qrow[warp * 32u + src];
                    const uint64_t c = c0 + cc + j;
                    const long long cid = (long long)(p.cand_lo + c);
                    const uint32_t hv = __shfl_sync(kFullMask, have, src);
                    const float th = __shfl_sync(kFullMask, thr, src);
                    if (lane == src) maybe &= maybe - 1u;
                    // query src's sorted list, lane l holding entries l and l + 32 (read while the rows are fetched)
                    float *wl = p.part_cos + ((size_t)blockIdx.y * p.m + (q0 + warp * 32u + src)) * p.K;
                    long long *wi = p.part_ids + ((size_t)blockIdx.y * p.m + (q0 + warp * 32u + src)) * p.K;
                    float e0 = 0.f, e1 = 0.f;
                    long long i0 = -1, i1 = -1;
                    if (lane < hv) { e0 = __ldcg(wl + lane); i0 = __ldcg(wi + lane); }
                    if (lane + 32u < hv) { e1 = __ldcg(wl + lane + 32u); i1 = __ldcg(wi + lane + 32u); }
                    const float dot = warp_row_dot(T4, (size_t)qr, (size_t)(p.cand_lo + c), p.d4, p.ld4, lane);
                    const float cs = dot * __shfl_sync(kFullMask, qinv, src) * __shfl_sync(kFullMask, icv, j);
                    if (!(cs > p.tau) || cid == qr || (hv == p.K && cs < th)) continue;     // same for every lane
                    const bool a0 = lane < hv && !ranks_ahead_tc(cs, cid, e0, i0);         // entries that stay ahead: a prefix
                    const bool a1 = lane + 32u < hv && !ranks_ahead_tc(cs, cid, e1, i1);
                    const uint32_t pos = (uint32_t)__popc(__ballot_sync(kFullMask, a0)) + (uint32_t)__popc(__ballot_sync(kFullMask, a1));
                    const uint32_t km2 = p.K >= 2u ? p.K - 2u : 0u;
                    const float e_km2 = km2 < 32u ? __shfl_sync(kFullMask, e0, km2) : __shfl_sync(kFullMask, e1, km2 - 32u);
                    if (pos < p.K) {
                        if (lane < hv && !a0 && lane + 1u < p.K) { wl[lane + 1u] = e0; wi[lane + 1u] = i0; }
                        if (lane + 32u < hv && !a1 && lane + 33u < p.K) { wl[lane + 33u] = e1; wi[lane + 33u] = i1; }
                        if (lane == 0) { wl[pos] = cs; wi[pos] = cid; }
                        if (lane == src) {
                            have = hv < p.K ? hv + 1u : p.K;
                            thr = have == p.K ? (pos == p.K - 1u ? cs : e_km2) : p.tau;
                        }
                    }
                    __syncwarp();
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(tempty + b);                              // this accumulator buffer may be overwritten
        }
    } else if (warp == 4) {
        // ================= MMA issue: one lane =================
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(kTcN >> 3) << 17) | ((uint32_t)(kTcM >> 4) << 24);
            // the query block: one bulk copy per K-block, all on one barrier
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         ::"r"(smem_addr(afull)), "r"(nkb * (uint32_t)kScABlock) : "memory");
            for (uint32_t kb = 0; kb < nkb; ++kb)
                bulk_to_smem(a_op + (size_t)kb * kScABlock, p.qsplit + ((size_t)blockIdx.x * nkb + kb) * kScABlock,
                             (uint32_t)kScABlock, afull);
            bool ok = mbar_wait(afull, 0u, abort_flag);
            uint64_t g = 0;
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
                    const uint32_t abase = smem_addr(a_op + (size_t)kb * kScABlock);
                    const uint32_t bbase = smem_addr(b_op + (size_t)s * kScStageBytes);
                    const uint32_t chunks = p.d4 - kb * 8u < 8u ? p.d4 - kb * 8u : 8u;   // 16-byte chunks with data
                    const uint32_t nk = (chunks + 1u) / 2u;                              // MMAs of K = 8 columns
                    for (uint32_t kk = 0; kk < nk; ++kk) {
                        const uint64_t qa = umma_desc(abase + 2 * kk * kScAChunk, kScAChunk, 128);
                        const uint64_t cb = umma_desc(bbase + 2 * kk * kTcChunkStrideC, kTcChunkStrideC, 128);
                        umma_tf32(dst, qa, cb, idesc, (kb | kk) ? 1u : 0u);
                    }
                    umma_commit(empty + s);                       // the stage is free once these MMAs have read it
                }
                if (ok) umma_commit(tfull + b);                   // the tile's accumulator is complete
            }
        } else if (lane == 1) {
            // Relay.  More loader groups than stages take turns on a stage, and a parity wait cannot
            // tell "free again" from "free two uses ago"; this lane waits for every release in order
            // and publishes the count, which the loaders poll.
            const uint64_t total_g = n_tiles * nkb;
            for (uint64_t g = 0; g < total_g; ++g) {
                const uint32_t s = (uint32_t)(g % kTcStages);
                const uint64_t use = g / kTcStages;
                if (!mbar_wait(empty + s, (uint32_t)(use & 1), abort_flag)) break;
                __threadfence_block();
                consumed[s] = (uint32_t)(use + 1);
            }
        }
    } else {
        // ================= loaders: candidate rows as they are =================
        const uint32_t group = (tid - 5 * 32) / kTcLoaders, ltid = (tid - 5 * 32) % kTcLoaders;
        const uint64_t total_g = n_tiles * nkb;
        float4 x[kTcPer];
        uint64_t g = group;
        if (g < total_g) candidates_issue(p, x, (uint32_t)(g % nkb) * kTcKB, ltid, (t_lo + g / nkb) * kTcN, nc);
        while (g < total_g) {
            const uint32_t s = (uint32_t)(g % kTcStages);
            {   // the stage's previous use must have been read by the MMAs
                const uint32_t need = (uint32_t)(g / kTcStages);
                bool ok = false;
                for (uint32_t spin = 0; spin < kTcSpinLimit * 16u; ++spin) {
                    if (consumed[s] >= need) { ok = true; break; }
                    if ((spin & 1023u) == 1023u && *abort_flag) break;
                }
                if (!ok) { *abort_flag = 1; break; }
                __threadfence_block();
            }
            unsigned char *st = b_op + (size_t)s * kScStageBytes;
#pragma unroll
            for (int it = 0; it < kTcPer; ++it) {
                const uint32_t e = ltid + it * kTcLoaders;
                *reinterpret_cast<float4 *>(st + (e & 7) * kTcChunkStrideC + (e >> 3) * 16) = x[it];
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");         // stores -> tensor-core reads
            mbar_arrive(full + s);
            g += kScGroups;
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

static size_t topk_screen_smem_bytes()
{
    return (size_t)kScMaxKB * kScABlock + (size_t)kTcStages * kScStageBytes + (2 * kTcStages + 5) * 8 + 16 + kTcM * 8 + 128;
}

bool topk_screen_fits(uint32_t d) { return (d + kTcKB - 1) / kTcKB <= (uint32_t)kScMaxKB; }

size_t topk_tc_smem_bytes()
{
    return (size_t)kTcStages * kTcStageBytes + (2 * kTcStages + 4) * 8 + 16 + kTcM * 8 + 8 * kTcN * 4 + 128;
}

// Returns the launches made, or -1 on a launch error.  Results go to part_* ([splits][m][K]); the caller merges.
size_t topk_tc_qsplit_bytes(uint64_t m, uint32_t d)
{
    const uint64_t qblocks = (m + kTcM - 1) / kTcM, nkb = (d + kTcKB - 1) / kTcKB;
    return (size_t)(qblocks * nkb * 2 * kTcOperand);          // the screening layout needs less (kScABlock per K-block)
}

int launch_topk_tc(const float *table, uint32_t d, uint32_t ld, uint64_t vocab, const long long *queries, uint64_t m,
                   uint64_t cand_lo, uint64_t cand_hi, uint32_t K, float tau, const float *inv_norm,
                   unsigned char *qsplit, float *part_cos, long long *part_ids, uint32_t splits, int *error,
                   bool screen, cudaStream_t s)
{
    if (m == 0) return 0;
    const uint32_t nkb = (d + kTcKB - 1) / kTcKB;
    const unsigned qblocks = (unsigned)((m + kTcM - 1) / kTcM);
    screen = screen && topk_screen_fits(d);
    if (screen) topk_round_queries_kernel<<<qblocks * nkb, 256, 0, s>>>(table, queries, m, vocab, d / 4, ld / 4, nkb, qsplit);
    else topk_split_queries_kernel<<<qblocks * nkb, 256, 0, s>>>(table, queries, m, vocab, d / 4, ld / 4, nkb, qsplit);
    if (cudaGetLastError() != cudaSuccess) return -1;
    TcParams p;
    p.qsplit = qsplit;
    p.table = table; p.queries = queries; p.inv_norm = inv_norm; p.part_cos = part_cos; p.part_ids = part_ids;
    p.error = error; p.m = m; p.vocab = vocab; p.cand_lo = cand_lo; p.cand_hi = cand_hi;
    p.d4 = d / 4; p.ld4 = ld / 4; p.K = K; p.splits = splits; p.tau = tau;
    dim3 grid((unsigned)((m + kTcM - 1) / kTcM), splits);
    if (screen) {
        const size_t sm = topk_screen_smem_bytes();
        if (cudaFuncSetAttribute(topk_cosine_screen_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess)
            return -1;
        topk_cosine_screen_kernel<<<grid, kScThreads, sm, s>>>(p);
    } else {
        const size_t sm = topk_tc_smem_bytes();
        if (cudaFuncSetAttribute(topk_cosine_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess)
            return -1;
        topk_cosine_tc_kernel<<<grid, kTcThreads, sm, s>>>(p);
    }
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 2;
}

}  // namespace w2v

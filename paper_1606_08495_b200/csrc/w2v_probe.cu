// Memory-system ceilings for the access patterns of the update kernels, measured on the model's own
// output table: random rows gathered (and optionally added to) with the same row layout, loads,
// reductions and rows in flight per warp as the step, but with precomputable row numbers and no
// sampling or arithmetic in the way.  What the step kernels reach is judged against these figures
// rather than against a plain copy.  The additions add +0.0f, so the table's values do not change.
#include "../../include/w2v.h"
#include "w2v_device.cuh"
#include "w2v_internal.h"

namespace w2v {

namespace {

constexpr int kProbeTB = 4;            // rows in flight per warp, as in the step kernels at d = 300

// row number of the i-th access: a mixing hash of i, reduced to [0, span)
__device__ __forceinline__ uint32_t probe_row(unsigned long long i, uint32_t span, uint32_t salt)
{
    unsigned long long x = (i + 1ull) * 0x9E3779B97F4A7C15ull + salt;
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return (uint32_t)(x % span);
}

template <int VPL, uint32_t access>
__global__ void __launch_bounds__(kBlock, 2)
probe_rows_kernel(float *V, const uint2 *alias, uint32_t vocab, uint32_t d4, uint32_t ld4, uint32_t span,
                  unsigned long long per_warp, uint32_t zero, float *sink)
{
    constexpr int NCH = (VPL + 3) / 4;
    const uint32_t lane = threadIdx.x & 31;
    const unsigned long long warp = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    float4 *V4 = reinterpret_cast<float4 *>(V);
    constexpr bool with_alias = access == W2V_PROBE_GATHER_ALIAS || access == W2V_PROBE_GATHER_RED_ALIAS;
    constexpr bool with_red = access == W2V_PROBE_GATHER_RED || access == W2V_PROBE_GATHER_RED_ALIAS ||
                          access == W2V_PROBE_TOUCH_RED;
    float acc = 0.f;
    for (unsigned long long base = 0; base < per_warp; base += 32) {
        // 32 row numbers per round, one per lane; with_alias: each goes through one random 8-byte
        // read of the alias table first (what a negative draw costs)
        uint32_t mine = probe_row(warp * per_warp + base + lane, span, 0u);
        if (with_alias) {
            const uint2 e = __ldg(alias + probe_row(warp * per_warp + base + lane, vocab, 77u));
            if (e.x == 0u && e.y == 0xFFFFFFFFu) mine = 0u;          // never true for a built table
        }
        for (uint32_t j = 0; j < 32; j += kProbeTB) {
            uint32_t r[kProbeTB];
            Row<VPL> v[kProbeTB];
            uint32_t x[kProbeTB][NCH];
#pragma unroll
            for (int t = 0; t < kProbeTB; ++t) {
                r[t] = __shfl_sync(kFullMask, mine, j + t);
                if (access == W2V_PROBE_TOUCH_RED) {
                    row_touch<NCH>(x[t], V4 + (size_t)r[t] * ld4, d4, lane);
                    row_zero(v[t]);
                } else {
                    row_load(v[t], V4 + (size_t)r[t] * ld4, d4, lane);
                }
            }
#pragma unroll
            for (int t = 0; t < kProbeTB; ++t) {
                uint32_t off = 0u;
                float s = 0.f;
                if (access == W2V_PROBE_TOUCH_RED) {
                    off = touch_fence<NCH>(x[t], zero);
                } else {
                    Row<VPL> one;
#pragma unroll
                    for (int k = 0; k < VPL; ++k) one.x[k] = make_float4(1.f, 1.f, 1.f, 1.f);
                    s = warp_sum(row_dot_partial(one, v[t]));
                    acc += s;
                }
                if (with_red) {
                    Row<VPL> z;
                    row_zero(z);
                    // the factor depends on the gathered row, so the addition cannot be issued before it arrived
                    row_red_scaled(V4 + (size_t)r[t] * ld4 + off, s * 0.0f, z, d4, lane);
                }
            }
        }
    }
    if (acc == 12345.678f) *sink = acc;
}

// ---- ring of bulk copies: how fast one SM can pull L2-resident bytes into shared memory -----------
// One block per SM; `producers` lanes (one per warp) issue cp.async.bulk copies of `stage_bytes` into a
// ring of `stages` slots, each on the slot's "full" barrier once a consumer lane has released the slot;
// the consumer lane does nothing but wait for "full" and arrive on "empty".  Every block reads the same
// stream (as the blocks of one candidate split of the retrieval kernels do), so after the first pass the
// source sits in L2.  Waits are bounded; a block that gives up raises *error.
__device__ __forceinline__ uint32_t probe_saddr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool probe_try(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(probe_saddr(bar)), "r"(parity) : "memory");
    return done != 0;
}
__device__ __forceinline__ bool probe_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    for (uint32_t spin = 0; spin < (1u << 24); ++spin) {
        if (probe_try(bar, parity)) return true;
        if ((spin & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

__global__ void __launch_bounds__(256, 1)
probe_bulk_ring_kernel(const unsigned char *src, unsigned long long span, uint32_t stage_bytes, uint32_t stages,
                       uint32_t copies, uint32_t producers, int *error)
{
    extern __shared__ __align__(128) unsigned char probe_smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(probe_smem + (size_t)stage_bytes * stages);     // [stages] (full, empty)
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        abort_word = 0;
        for (uint32_t i = 0; i < 2 * stages; ++i)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(probe_saddr(bars + i)), "r"(1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (lane == 0 && warp < producers) {
        unsigned long long off = ((unsigned long long)warp * stage_bytes) % span;
        for (uint32_t g = warp; g < copies; g += producers) {
            const uint32_t s = g % stages;
            uint64_t *full = bars + 2 * s, *empty = full + 1;
            if (!probe_wait(empty, ((g / stages) & 1) ^ 1, abort_flag)) break;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(probe_saddr(full)), "r"(stage_bytes) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(probe_saddr(probe_smem + (size_t)s * stage_bytes)), "l"(src + off), "r"(stage_bytes), "r"(probe_saddr(full)) : "memory");
            off += (unsigned long long)stage_bytes * producers;
            if (off + stage_bytes > span) off = ((unsigned long long)warp * stage_bytes) % span;
        }
    } else if (lane == 0 && warp == producers) {
        uint32_t g = 0;
        for (; g < copies; ++g) {
            const uint32_t s = g % stages;
            uint64_t *full = bars + 2 * s, *empty = full + 1;
            if (!probe_wait(full, (g / stages) & 1, abort_flag)) break;
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(probe_saddr(empty)) : "memory");
        }
        if (g < copies) {
            // giving up: copies already issued may still land; give them their time before shared memory goes away
            for (uint32_t j = g; j < g + stages && j < copies; ++j)
                for (uint32_t spin = 0; spin < (1u << 20); ++spin)
                    if (probe_try(bars + 2 * (j % stages), (j / stages) & 1)) break;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && abort_word) atomicExch(error, 4);
}

// ---- producer, ring and MMA issuer coupled, without an epilogue ------------------------------------
// What the retrieval screen's feed can reach at best: one block per SM with an 80 KB query operand in
// shared memory, a ring of `stages` slots of `kps` K-blocks (16 KB each, 10 per 256-candidate tile), two
// producer lanes issuing one bulk copy per slot, and one lane issuing the tile's 19 bf16 MMAs
// (128 x 256 x 16) from the slots and committing each slot's "empty" barrier.  Nobody reads the two
// accumulators.  span_tiles = 1: a slot holds the next kps K-blocks whichever tile they belong to;
// 0: slots do not span tiles (the tile's last slot is short).  Groups of 64 blocks read the same stream,
// as the blocks of one candidate split do.  The operands are whatever bytes the table holds, read as
// bf16: only the timing is of interest.  Waits are bounded; a block that gives up raises *error.
constexpr int kRingA = 10 * 4 * 128 * 16;               // the query operand: 10 K-blocks x 4 chunks x 128 rows x 16 B
constexpr int kRingKB = 4 * 256 * 16;                   // one K-block of a candidate tile
__device__ long long g_probe_cycles[2];                 // block 0: cycles of the MMA lane's loop, cycles it waited for data

__device__ __forceinline__ uint64_t probe_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
__device__ __forceinline__ void probe_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}\n"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0), "r"(0), "r"(0), "r"(0) : "memory");
}
__device__ __forceinline__ void probe_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(probe_saddr(bar)) : "memory");
}

__global__ void __launch_bounds__(128, 1)
probe_mma_ring_kernel(const unsigned char *src, unsigned long long stream_stride, uint32_t kps, uint32_t stages, uint32_t tiles,
                      uint32_t span_tiles, int *error)
{
    extern __shared__ __align__(128) unsigned char probe_smem[];
    unsigned char *As = probe_smem, *Bs = probe_smem + kRingA;
    const uint32_t stage_bytes = kps * (uint32_t)kRingKB;
    uint64_t *full = reinterpret_cast<uint64_t *>(Bs + (size_t)stages * stage_bytes), *empty = full + stages, *done = empty + stages;
    uint32_t *slot = reinterpret_cast<uint32_t *>(done + 1);
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;
    const uint32_t tid = threadIdx.x, warp = tid >> 5;
    const unsigned char *stream = src + (unsigned long long)(blockIdx.x / 64u) * stream_stride;
    for (uint32_t i = tid; i < (uint32_t)kRingA / 16u; i += 128) reinterpret_cast<uint4 *>(As)[i] = reinterpret_cast<const uint4 *>(stream)[i];
    if (tid == 0) {
        abort_word = 0;
        for (uint32_t i = 0; i < 2 * stages + 1; ++i)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(probe_saddr(full + i)), "r"(1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(probe_saddr(slot)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");         // the operand was written by ordinary stores
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tm = *slot;
    const uint32_t nkb = 10, total_kb = tiles * nkb;
    const uint32_t spt = (nkb + kps - 1) / kps;                          // slots per tile when slots do not span tiles
    const uint32_t total_g = span_tiles ? (total_kb + kps - 1) / kps : tiles * spt;
    if (tid == 0) {
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint64_t a0 = probe_desc(probe_saddr(As), 128 * 16, 128), b0 = probe_desc(probe_saddr(Bs), 256 * 16, 128);
        constexpr uint64_t aS = (2 * 128 * 16) >> 4, bS = (2 * 256 * 16) >> 4;
        long long waited = 0;
        const long long t0 = clock64();
        uint32_t s = 0, ph = 0, kb = 0, tile = 0;
        bool ok = true;
        for (uint32_t g = 0; g < total_g; ++g) {
            const long long w0 = clock64();
            ok = probe_wait(full + s, ph, abort_flag);
            if (!ok) break;
            waited += clock64() - w0;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t cnt = span_tiles ? (total_kb - g * kps < kps ? total_kb - g * kps : kps) : (nkb - kb < kps ? nkb - kb : kps);
            uint64_t cb = b0 + (uint64_t)s * (stage_bytes >> 4);
            for (uint32_t j = 0; j < cnt; ++j) {
                const uint32_t d = tm + (tile & 1u) * 256u;
                probe_mma(d, a0 + kb * 2 * aS, cb, idesc, kb ? 1u : 0u);
                if (kb + 1 < nkb) probe_mma(d, a0 + kb * 2 * aS + aS, cb + bS, idesc, 1u);     // the tile's last K-block: one k-step of data
                cb += 2 * bS;
                if (++kb == nkb) { kb = 0; ++tile; }
            }
            probe_commit(empty + s);
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
        const long long t1 = clock64();
        probe_commit(done);                                               // every MMA has completed before tensor memory is released
        if (ok) probe_wait(done, 0u, abort_flag);
        if (blockIdx.x == 0) { g_probe_cycles[0] = t1 - t0; g_probe_cycles[1] = waited; }
    } else if (tid == 32 || tid == 64) {
        // Stages alternate between the two lanes.  With two or more slots a lane that has passed its wait for
        // slot use u - 1 has thereby seen every earlier release of that slot, so the parity it waits on next
        // cannot be mistaken for an older phase.
        const uint32_t w = tid == 32 ? 0u : 1u;
        uint32_t g = w;
        for (; g < total_g; g += 2) {
            const uint32_t s = g % stages;
            if (!probe_wait(empty + s, ((g / stages) & 1u) ^ 1u, abort_flag)) break;
            uint32_t kb_first, cnt;
            if (span_tiles) { kb_first = g * kps; cnt = total_kb - kb_first < kps ? total_kb - kb_first : kps; }
            else { const uint32_t t = g / spt, st = g - t * spt; kb_first = t * nkb + st * kps; cnt = nkb - st * kps < kps ? nkb - st * kps : kps; }
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(probe_saddr(full + s)), "r"(cnt * (uint32_t)kRingKB) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(probe_saddr(Bs + (size_t)s * stage_bytes)), "l"(stream + (unsigned long long)kb_first * kRingKB),
                           "r"(cnt * (uint32_t)kRingKB), "r"(probe_saddr(full + s)) : "memory");
        }
        // this lane's copies still in flight land before shared memory goes away
        for (uint32_t back = 2; back <= stages + 1u && back <= g; back += 2) {
            const uint32_t j = g - back;
            for (uint32_t spin = 0; spin < (1u << 20); ++spin)
                if (probe_try(full + j % stages, (j / stages) & 1u)) break;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0 && abort_word) atomicExch(error, 4);
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(512));
    }
}

}  // namespace

int launch_probe_bulk_ring(const unsigned char *src, unsigned long long span, uint32_t stage_bytes, uint32_t stages,
                           uint32_t copies, uint32_t producers, int *error, int sms, cudaStream_t s)
{
    const size_t sm = (size_t)stage_bytes * stages + 16 * (size_t)stages;
    if (cudaFuncSetAttribute(probe_bulk_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess) return -1;
    probe_bulk_ring_kernel<<<sms, 256, sm, s>>>(src, span, stage_bytes, stages, copies, producers, error);
    return cudaGetLastError() != cudaSuccess ? -1 : 1;
}

int launch_probe_mma_ring(const unsigned char *src, unsigned long long stream_stride, uint32_t kps, uint32_t stages, uint32_t tiles,
                          uint32_t span_tiles, int *error, int sms, cudaStream_t s)
{
    const size_t sm = (size_t)kRingA + (size_t)stages * kps * kRingKB + 16 * (size_t)stages + 64;
    if (cudaFuncSetAttribute(probe_mma_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm) != cudaSuccess) return -1;
    probe_mma_ring_kernel<<<sms, 128, sm, s>>>(src, stream_stride, kps, stages, tiles, span_tiles, error);
    return cudaGetLastError() != cudaSuccess ? -1 : 1;
}

// cycles of block 0's MMA lane (whole loop, and the part spent waiting for data); call after the stream has been synchronised
int read_probe_mma_ring(long long *cycles, long long *waited)
{
    long long v[2];
    if (cudaMemcpyFromSymbol(v, g_probe_cycles, sizeof v) != cudaSuccess) return -1;
    *cycles = v[0]; *waited = v[1];
    return 0;
}

int launch_probe_rows(float *V, const uint2 *alias, uint32_t vocab, uint32_t d4, uint32_t ld4, uint32_t span,
                      unsigned long long rows, uint32_t access, float *sink, int sms, cudaStream_t s,
                      unsigned long long *rows_done)
{
    const int grid = sms * 2;
    const unsigned long long warps = (unsigned long long)grid * (kBlock / 32);
    unsigned long long per_warp = (rows + warps - 1) / warps;
    per_warp = (per_warp + 31) / 32 * 32;
    *rows_done = per_warp * warps;
#define CALL_PROBE(VPL)                                                                                          \
    switch (access) {                                                                                            \
        case W2V_PROBE_GATHER: probe_rows_kernel<VPL, W2V_PROBE_GATHER><<<grid, kBlock, 0, s>>>(V, alias, vocab, d4, ld4, span, per_warp, 0u, sink); break; \
        case W2V_PROBE_GATHER_RED: probe_rows_kernel<VPL, W2V_PROBE_GATHER_RED><<<grid, kBlock, 0, s>>>(V, alias, vocab, d4, ld4, span, per_warp, 0u, sink); break; \
        case W2V_PROBE_GATHER_ALIAS: probe_rows_kernel<VPL, W2V_PROBE_GATHER_ALIAS><<<grid, kBlock, 0, s>>>(V, alias, vocab, d4, ld4, span, per_warp, 0u, sink); break; \
        case W2V_PROBE_GATHER_RED_ALIAS: probe_rows_kernel<VPL, W2V_PROBE_GATHER_RED_ALIAS><<<grid, kBlock, 0, s>>>(V, alias, vocab, d4, ld4, span, per_warp, 0u, sink); break; \
        default: probe_rows_kernel<VPL, W2V_PROBE_TOUCH_RED><<<grid, kBlock, 0, s>>>(V, alias, vocab, d4, ld4, span, per_warp, 0u, sink); break; \
    }
    switch ((d4 + 31) / 32) {
        case 1: CALL_PROBE(1); break;
        case 2: CALL_PROBE(2); break;
        case 3: CALL_PROBE(3); break;
        case 4: CALL_PROBE(4); break;
        default: return -2;
    }
#undef CALL_PROBE
    return cudaGetLastError() != cudaSuccess ? -1 : 1;
}

}  // namespace w2v

// Integer half of the step: sub-sampling, compaction ("dirty" contexts, footnote to
// Section 3), window radii, pair offsets and the explicit pair list of Algorithm 3
// (W_input, W_output) with the negatives of Algorithms 1 and 2.
#include "w2v_sample.cuh"

namespace w2v {

enum : uint8_t { kFlagKept = 1, kFlagSentinel = 2 };

// ---- pass 1: classify every token, count per tile --------------------------------
__global__ void __launch_bounds__(kScanBlock)
classify_kernel(const int32_t *__restrict__ tokens, uint64_t n, SampleTables tab, uint32_t vocab,
                uint32_t k0, uint32_t k1, uint32_t step_lo, uint8_t *__restrict__ flags,
                uint2 *__restrict__ tile_sums, DevState *st)
{
    __shared__ uint32_t sh[33];
    const uint64_t base = (uint64_t)blockIdx.x * kScanTile + (uint64_t)threadIdx.x * kScanItems;
    uint32_t kept = 0, sent = 0, oov = 0;
#pragma unroll
    for (int e = 0; e < kScanItems; ++e) {
        const uint64_t i = base + e;
        if (i >= n) break;
        const int32_t w = tokens[i];
        uint8_t f = 0;
        if (w == -1) {
            f = kFlagSentinel; ++sent;
        } else if (w < 0 || (uint32_t)w >= vocab) {
            ++oov;
        } else {
            const uint32_t thr = __ldg(tab.keep_thr + w);
            bool keep = true;
            if (thr != 0xFFFFFFFFu)
                keep = philox4x32_10(k0, k1, (uint32_t)i, step_lo, kPurSubsample, 0).x < thr;
            if (keep) { f = kFlagKept; ++kept; }
        }
        flags[i] = f;
    }
    // pack the two counts (each <= 2048 per tile) into one word for a single block sum
    uint32_t total;
    block_exclusive_scan<uint32_t>(kept | (sent << 16), sh, total);
    if (threadIdx.x == 0) tile_sums[blockIdx.x] = make_uint2(total & 0xFFFFu, total >> 16);
    const uint32_t o = warp_sum(oov);
    if ((threadIdx.x & 31) == 0 && o) {
        atomicAdd(&st->oov, (unsigned long long)o);
        atomicOr(&st->status, 1u);
    }
}

// ---- pass 2: exclusive scan of the tile sums (one block) ---------------------------
__global__ void __launch_bounds__(1024)
scan_tiles_kernel(const uint2 *__restrict__ tile_sums, uint2 *__restrict__ tile_offs, uint32_t n_tiles,
                  DevState *st)
{
    __shared__ unsigned long long sh[33];
    unsigned long long carry = 0;   // kept in the low 32 bits, sentinels in the high 32 bits
    for (uint32_t b0 = 0; b0 < n_tiles; b0 += blockDim.x) {
        const uint32_t b = b0 + threadIdx.x;
        unsigned long long x = 0;
        if (b < n_tiles) {
            const uint2 s = tile_sums[b];
            x = (unsigned long long)s.x | ((unsigned long long)s.y << 32);
        }
        unsigned long long total;
        const unsigned long long ex = block_exclusive_scan<unsigned long long>(x, sh, total) + carry;
        if (b < n_tiles) tile_offs[b] = make_uint2((uint32_t)ex, (uint32_t)(ex >> 32));
        carry += total;
    }
    if (threadIdx.x == 0) {
        st->n_kept = carry & 0xFFFFFFFFull;
        st->n_sent = carry >> 32;
    }
}

// ---- pass 3: scatter the kept tokens ----------------------------------------------
__global__ void __launch_bounds__(kScanBlock)
scatter_kernel(const int32_t *__restrict__ tokens, uint64_t n, const uint8_t *__restrict__ flags,
               const uint2 *__restrict__ tile_offs, int32_t *__restrict__ ctok,
               uint32_t *__restrict__ cidx, uint32_t *__restrict__ csent)
{
    __shared__ uint32_t sh[33];
    const uint64_t base = (uint64_t)blockIdx.x * kScanTile + (uint64_t)threadIdx.x * kScanItems;
    uint8_t f[kScanItems];
    uint32_t kept = 0, sent = 0;
#pragma unroll
    for (int e = 0; e < kScanItems; ++e) {
        const uint64_t i = base + e;
        f[e] = i < n ? flags[i] : 0;
        kept += f[e] & kFlagKept;
        sent += (f[e] & kFlagSentinel) >> 1;
    }
    uint32_t total;
    const uint32_t ex = block_exclusive_scan<uint32_t>(kept | (sent << 16), sh, total);
    const uint2 off = tile_offs[blockIdx.x];
    uint32_t pos = off.x + (ex & 0xFFFFu);
    uint32_t sid = off.y + (ex >> 16);
#pragma unroll
    for (int e = 0; e < kScanItems; ++e) {
        if (f[e] & kFlagKept) {
            const uint64_t i = base + e;
            ctok[pos] = tokens[i];
            cidx[pos] = (uint32_t)i;
            csent[pos] = sid;
            ++pos;
        }
        sid += (f[e] & kFlagSentinel) >> 1;
    }
}

// ---- windows: radius b in 1..window per centre, clipped to its sentence ------------
__global__ void __launch_bounds__(256)
window_kernel(const uint32_t *__restrict__ cidx, const uint32_t *__restrict__ csent, uint32_t window,
              uint32_t k0, uint32_t k1, uint32_t step_lo, uint32_t il_phase, uint32_t il_stride,
              uint16_t *__restrict__ win, DevState *st)
{
    const uint32_t nk = (uint32_t)st->n_kept;
    const uint32_t q = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t cnt = 0;
    if (q < nk) {
        const uint32_t i = cidx[q];
        const uint32_t r = philox4x32_10(k0, k1, i, step_lo, kPurRadius, 0).x;
        // interleaved minibatches: only tokens with index = phase (mod stride) are input words of
        // this call; the others keep an empty window and serve as contexts only
        const uint32_t b = (il_stride > 1u && i % il_stride != il_phase) ? 0u : 1u + __umulhi(r, window);
        const uint32_t sid = csent[q];
        uint32_t left = 0, right = 0;
        while (left < b && q >= left + 1u && csent[q - left - 1u] == sid) ++left;
        while (right < b && q + right + 1u < nk && csent[q + right + 1u] == sid) ++right;
        win[q] = (uint16_t)(left | (right << 8));
        cnt = left + right;
    }
    const uint32_t pairs = warp_sum(cnt);
    const uint32_t centres = __popc(__ballot_sync(kFullMask, cnt > 0));
    if ((threadIdx.x & 31) == 0 && pairs) {
        atomicAdd(&st->pairs, (unsigned long long)pairs);
        atomicAdd(&st->centres, (unsigned long long)centres);
    }
}

// ---- pair offsets: exclusive scan of the context counts ------------------------------
__device__ __forceinline__ uint32_t win_count(uint16_t w, bool examples)
{
    return examples ? (w != 0 ? 1u : 0u) : (w & 0xFFu) + (w >> 8);
}

__global__ void __launch_bounds__(kScanBlock)
pair_tile_sums_kernel(const uint16_t *__restrict__ win, unsigned long long *__restrict__ cnt_tile,
                      const DevState *st, bool examples)
{
    __shared__ uint32_t sh[33];
    const uint32_t nk = (uint32_t)st->n_kept;
    const uint64_t base = (uint64_t)blockIdx.x * kScanTile + (uint64_t)threadIdx.x * kScanItems;
    uint32_t s = 0;
#pragma unroll
    for (int e = 0; e < kScanItems; ++e)
        if (base + e < nk) s += win_count(win[base + e], examples);
    uint32_t total;
    block_exclusive_scan<uint32_t>(s, sh, total);
    if (threadIdx.x == 0) cnt_tile[blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024)
pair_scan_tiles_kernel(unsigned long long *__restrict__ cnt_tile, uint32_t n_tiles)
{
    __shared__ unsigned long long sh[33];
    unsigned long long carry = 0;
    for (uint32_t b0 = 0; b0 < n_tiles; b0 += blockDim.x) {
        const uint32_t b = b0 + threadIdx.x;
        const unsigned long long x = b < n_tiles ? cnt_tile[b] : 0ull;
        unsigned long long total;
        const unsigned long long ex = block_exclusive_scan<unsigned long long>(x, sh, total) + carry;
        if (b < n_tiles) cnt_tile[b] = ex;
        carry += total;
    }
}

__global__ void __launch_bounds__(kScanBlock)
pair_offsets_kernel(const uint16_t *__restrict__ win, const unsigned long long *__restrict__ cnt_tile,
                    unsigned long long *__restrict__ pair_off, const DevState *st, bool examples)
{
    __shared__ uint32_t sh[33];
    const uint32_t nk = (uint32_t)st->n_kept;
    const uint64_t base = (uint64_t)blockIdx.x * kScanTile + (uint64_t)threadIdx.x * kScanItems;
    uint32_t c[kScanItems];
    uint32_t s = 0;
#pragma unroll
    for (int e = 0; e < kScanItems; ++e) {
        c[e] = base + e < nk ? win_count(win[base + e], examples) : 0u;
        s += c[e];
    }
    uint32_t total;
    uint32_t ex = block_exclusive_scan<uint32_t>(s, sh, total);
    unsigned long long off = cnt_tile[blockIdx.x] + ex;
#pragma unroll
    for (int e = 0; e < kScanItems; ++e) {
        if (base + e < nk) pair_off[base + e] = off;
        off += c[e];
    }
}

// ---- explicit pair list ----------------------------------------------------------------
__global__ void __launch_bounds__(kBlock)
emit_pairs_kernel(StepParams p, int32_t *__restrict__ centre, int32_t *__restrict__ context,
                  int32_t *__restrict__ negs, uint64_t cap)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    uint32_t draws = 0, redraws = 0;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, right = w >> 8;
        if (left + right == 0) continue;
        const int32_t c = p.ctok[q];
        const uint32_t i = p.cidx[q];
        unsigned long long pi = p.pair_off[q];
        for (uint32_t pp = q - left; pp <= q + right; ++pp) {
            if (pp == q) continue;
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            const uint32_t slot = pp + p.window - q;
            uint32_t n0, n1;
            draw_pair_negatives(p, i, slot, w_out, lane, n0, n1, draws, redraws);
            if (pi < cap) {
                if (lane == 0) { centre[pi] = c; context[pi] = (int32_t)w_out; }
                if (lane < p.negatives) negs[pi * p.negatives + lane] = (int32_t)n0;
                if (lane + 32u < p.negatives) negs[pi * p.negatives + lane + 32u] = (int32_t)n1;
            }
            ++pi;
        }
    }
    flush_draw_counts(p.st, draws, redraws);
}

// ---- the step's negatives as a list ---------------------------------------------------------
// negs[pair * N + k] for every pair of the chunk, pairs numbered as in the pair list.  A draw is a
// dependent chain (generator, one random 8-byte read of the alias table, compare); inside an update
// kernel that chain sits in front of every pair's row gathers with N of 32 lanes busy.  Here the
// lanes of a warp share out all cnt * N draws of a centre, so every lane has a draw in flight.
__global__ void __launch_bounds__(kBlock)
draw_negatives_kernel(StepParams p, int32_t *__restrict__ negs)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    const uint32_t N = p.negatives;
    uint32_t draws = 0, redraws = 0;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, cnt = left + (w >> 8);
        if (cnt == 0) continue;
        const uint32_t i = p.cidx[q];
        int32_t *dst = negs + p.pair_off[q] * N;
        const uint32_t items = cnt * N;
        for (uint32_t it = lane; it < items; it += 32) {
            const uint32_t j = it / N, k = it - j * N;
            const uint32_t pp = q - left + j + (j >= left ? 1u : 0u);      // position of the centre's j-th context
            const uint32_t w_out = (uint32_t)p.ctok[pp];
            dst[it] = (int32_t)draw_negative(p.tab.alias, p.vocab, p.k0, p.k1, i, p.step_lo, pp + p.window - q, k, w_out,
                                             draws, redraws);
        }
    }
    flush_draw_counts(p.st, draws, redraws);
}

// ---- small chunks: the whole integer half in one launch -------------------------------------
// A chunk of at most kSmallChunk tokens is classified, compacted and given its windows by a single
// block (the counters are cleared here too), so that a small step is two launches instead of six:
// with chunks this small the step is bound by launches, not by the GPU.
constexpr int kSmallBlock = 1024;
constexpr int kSmallItems = 8;

__global__ void __launch_bounds__(kSmallBlock)
sample_small_kernel(const int32_t *__restrict__ tokens, uint32_t n, SampleTables tab, uint32_t vocab, uint32_t k0,
                    uint32_t k1, uint32_t step_lo, uint32_t window, uint32_t il_phase, uint32_t il_stride,
                    int32_t *__restrict__ ctok, uint32_t *__restrict__ cidx, uint32_t *__restrict__ csent,
                    uint16_t *__restrict__ win, DevState *st)
{
    __shared__ uint32_t sh[33];
    __shared__ uint32_t s_pairs, s_centres, s_oov;
    const uint32_t base = threadIdx.x * kSmallItems;
    if (threadIdx.x == 0) { s_pairs = 0; s_centres = 0; s_oov = 0; }
    uint8_t f[kSmallItems];
    uint32_t kept = 0, sent = 0, oov = 0;
#pragma unroll
    for (int e = 0; e < kSmallItems; ++e) {
        const uint32_t i = base + e;
        f[e] = 0;
        if (i >= n) continue;
        const int32_t w = tokens[i];
        if (w == -1) {
            f[e] = kFlagSentinel; ++sent;
        } else if (w < 0 || (uint32_t)w >= vocab) {
            ++oov;
        } else {
            const uint32_t thr = __ldg(tab.keep_thr + w);
            bool keep = true;
            if (thr != 0xFFFFFFFFu) keep = philox4x32_10(k0, k1, i, step_lo, kPurSubsample, 0).x < thr;
            if (keep) { f[e] = kFlagKept; ++kept; }
        }
    }
    uint32_t total;
    const uint32_t ex = block_exclusive_scan<uint32_t>(kept | (sent << 16), sh, total);
    uint32_t pos = ex & 0xFFFFu, sid = ex >> 16;
#pragma unroll
    for (int e = 0; e < kSmallItems; ++e) {
        if (f[e] & kFlagKept) {
            const uint32_t i = base + e;
            ctok[pos] = tokens[i]; cidx[pos] = i; csent[pos] = sid;
            ++pos;
        }
        sid += (f[e] & kFlagSentinel) >> 1;
    }
    if (oov) atomicAdd(&s_oov, oov);
    __syncthreads();                                   // the compacted chunk is complete (block-wide)
    const uint32_t nk = total & 0xFFFFu;
    uint32_t pairs = 0, centres = 0;
    for (uint32_t q = threadIdx.x; q < nk; q += kSmallBlock) {
        const uint32_t i = cidx[q];
        const uint32_t r = philox4x32_10(k0, k1, i, step_lo, kPurRadius, 0).x;
        const uint32_t b = (il_stride > 1u && i % il_stride != il_phase) ? 0u : 1u + __umulhi(r, window);
        const uint32_t sd = csent[q];
        uint32_t left = 0, right = 0;
        while (left < b && q >= left + 1u && csent[q - left - 1u] == sd) ++left;
        while (right < b && q + right + 1u < nk && csent[q + right + 1u] == sd) ++right;
        win[q] = (uint16_t)(left | (right << 8));
        pairs += left + right;
        centres += (left + right) ? 1u : 0u;
    }
    pairs = warp_sum(pairs); centres = warp_sum(centres);
    if ((threadIdx.x & 31) == 0 && pairs) { atomicAdd(&s_pairs, pairs); atomicAdd(&s_centres, centres); }
    __syncthreads();
    if (threadIdx.x == 0) {
        st->n_kept = nk; st->n_sent = total >> 16; st->centres = s_centres; st->pairs = s_pairs;
        st->neg_draws = 0; st->neg_redraws = 0; st->oov = s_oov; st->status = s_oov ? 1u : 0u; st->pad = 0;
    }
}

int launch_sample_small(const int32_t *tokens, uint64_t n, const SampleTables &tab, uint32_t vocab, uint32_t k0,
                        uint32_t k1, uint32_t step_lo, uint32_t window, uint32_t il_phase, uint32_t il_stride,
                        const Scratch &sc, DevState *st, cudaStream_t s)
{
    sample_small_kernel<<<1, kSmallBlock, 0, s>>>(tokens, (uint32_t)n, tab, vocab, k0, k1, step_lo, window, il_phase,
                                                  il_stride, sc.ctok, sc.cidx, sc.csent, sc.win, st);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

// ---- launchers ---------------------------------------------------------------------------
static inline uint32_t tiles_for(uint64_t n) { return (uint32_t)((n + kScanTile - 1) / kScanTile); }

int launch_compact(const int32_t *tokens, uint64_t n, const SampleTables &tab, uint32_t vocab,
                   uint32_t k0, uint32_t k1, uint32_t step_lo, const Scratch &sc, DevState *st,
                   cudaStream_t s)
{
    const uint32_t nt = tiles_for(n);
    if (nt) {
        classify_kernel<<<nt, kScanBlock, 0, s>>>(tokens, n, tab, vocab, k0, k1, step_lo, sc.flags,
                                                  sc.tile_sums, st);
    }
    scan_tiles_kernel<<<1, 1024, 0, s>>>(sc.tile_sums, sc.tile_offs, nt, st);
    if (nt) {
        scatter_kernel<<<nt, kScanBlock, 0, s>>>(tokens, n, sc.flags, sc.tile_offs, sc.ctok, sc.cidx,
                                                 sc.csent);
    }
    if (cudaGetLastError() != cudaSuccess) return -1;
    return nt ? 3 : 1;
}

int launch_windows(uint64_t n, uint32_t window, uint32_t k0, uint32_t k1, uint32_t step_lo,
                   uint32_t il_phase, uint32_t il_stride, const Scratch &sc, DevState *st, cudaStream_t s)
{
    if (n == 0) return 0;
    const uint32_t nb = (uint32_t)((n + 255) / 256);
    window_kernel<<<nb, 256, 0, s>>>(sc.cidx, sc.csent, window, k0, k1, step_lo, il_phase, il_stride, sc.win,
                                     st);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

int launch_pair_offsets(uint64_t n, const Scratch &sc, DevState *st, cudaStream_t s, bool examples)
{
    const uint32_t nt = tiles_for(n);
    if (nt == 0) return 0;
    pair_tile_sums_kernel<<<nt, kScanBlock, 0, s>>>(sc.win, sc.cnt_tile, st, examples);
    pair_scan_tiles_kernel<<<1, 1024, 0, s>>>(sc.cnt_tile, nt);
    pair_offsets_kernel<<<nt, kScanBlock, 0, s>>>(sc.win, sc.cnt_tile, sc.pair_off, st, examples);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 3;
}

// centre[pair], context[pair] for every pair of the chunk (the word ids of the pair list, without the negatives)
__global__ void __launch_bounds__(kBlock)
pair_words_kernel(StepParams p, int32_t *__restrict__ centre, int32_t *__restrict__ context)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t nk = (uint32_t)p.st->n_kept;
    for (uint32_t q = warp; q < nk; q += nwarps) {
        const uint32_t w = p.win[q];
        const uint32_t left = w & 0xFFu, cnt = left + (w >> 8);
        if (cnt == 0) continue;
        const int32_t c = p.ctok[q];
        const unsigned long long pair0 = p.pair_off[q];
        for (uint32_t j = lane; j < cnt; j += 32) {
            centre[pair0 + j] = c;
            context[pair0 + j] = p.ctok[q - left + j + (j >= left ? 1u : 0u)];
        }
    }
}

int launch_draw_negatives(const StepParams &p, int32_t *negs, int grid, cudaStream_t s)
{
    draw_negatives_kernel<<<grid, kBlock, 0, s>>>(p, negs);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

// the whole pair list of a step for the passes that stream over it: two launches
int launch_pair_list(const StepParams &p, int32_t *centre, int32_t *context, int32_t *negs, int grid, cudaStream_t s)
{
    pair_words_kernel<<<grid, kBlock, 0, s>>>(p, centre, context);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return launch_draw_negatives(p, negs, grid, s) < 0 ? -1 : 2;
}

int launch_emit_pairs(const StepParams &p, int32_t *centre, int32_t *context, int32_t *negs,
                      uint64_t cap, int grid, cudaStream_t s)
{
    emit_pairs_kernel<<<grid, kBlock, 0, s>>>(p, centre, context, negs, cap);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

}  // namespace w2v

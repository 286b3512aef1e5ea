// Internal declarations of libw2v: device-side state, kernel parameter blocks and
// the host launchers each .cu file exports to the C-ABI layer.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace w2v {

// Counter layout of every random choice (key = seed, with the high word of the step
// number xor-ed into the high key word):
//   c0 = token index in the chunk (row number for initialisation)
//   c1 = low word of the step number (column/4 for initialisation)
//   c2 = purpose | slot << 8, slot = context position - centre position + window
//   c3 = k | attempt << 16 (k-th negative of the pair, attempt-th re-draw)

constexpr int kBlock = 256;            // threads per block of the update kernels
constexpr int kScanBlock = 256;        // threads per block of the compaction kernels
constexpr int kScanItems = 8;          // tokens per thread
constexpr int kScanTile = kScanBlock * kScanItems;
constexpr int kMaxRedraw = 16;

// Counters and results that live on the device during a step.
struct DevState {
    unsigned long long n_kept;
    unsigned long long n_sent;
    unsigned long long centres;
    unsigned long long pairs;
    unsigned long long neg_draws;
    unsigned long long neg_redraws;
    unsigned long long oov;
    unsigned int status;
    unsigned int pad;
};

struct SampleTables {
    const uint32_t *keep_thr;   // [vocab] keep iff thr == 2^32-1 or random word < thr
    const uint2 *alias;         // [vocab] .x = acceptance threshold, .y = alias
};

// Everything the kernels of one step need.
struct StepParams {
    float *U;
    float *V;
    SampleTables tab;
    // compacted chunk
    const int32_t *ctok;        // word id of kept token q
    const uint32_t *cidx;       // its index in the chunk (random counter c0)
    const uint16_t *win;        // contexts to the left (low byte) and right (high byte)
    DevState *st;
    uint32_t vocab;
    uint32_t d4;                // d / 4
    uint32_t ld4;               // row stride of U and V in float4 units (>= d4)
    uint32_t window;
    uint32_t negatives;
    uint32_t k0, k1;            // Philox key
    uint32_t step_lo;
    float lr;
    // snapshot mode / pair list
    const unsigned long long *pair_off;   // first pair index of centre q
    float *G;                   // [pairs * (1 + negatives)] coefficients
    float *DU;                  // [kept * d] per-centre sums of G v(target)
    // pair list of the step (column shards with narrow slices): written once, streamed by the passes
    const int32_t *l_centre;    // [pairs]
    const int32_t *l_context;   // [pairs]
    const int32_t *l_negs;      // [pairs * negatives]
    double *DV;                 // [hot_rows * d] fp64 sums of G u(c) for the most-hit output rows
    uint32_t hot_rows;          // output rows [0, hot_rows) accumulate in DV (snapshot mode)
    uint32_t zero;              // always 0; ANDed with a loaded word it ties a later address to that load's arrival
    uint32_t keep_negs;         // snapshot mode: the negatives of every pair are in l_negs (SGNS: drawn by a launch of their own before pass 1; CBOW: written by pass 1) and read back by the passes
};

// F arrays of all shards (this one included) that receive a shard's partial dot products.
constexpr int kMaxShards = 16;
constexpr uint32_t kNarrowD4 = 16;     // slices of at most this many float4 use the pair-list passes
struct ShardPeers {
    float *F[kMaxShards];
    uint32_t n;
};

// Epoch words of all shards (this one included) for the barrier of a peer-to-peer exchange.
struct PeerFlags {
    uint32_t *p[kMaxShards];
    uint32_t n;
};

struct Scratch {
    uint64_t n_cap = 0;
    uint8_t *flags = nullptr;
    uint2 *tile_sums = nullptr;
    uint2 *tile_offs = nullptr;
    int32_t *ctok = nullptr;
    uint32_t *cidx = nullptr;
    uint32_t *csent = nullptr;
    uint16_t *win = nullptr;
    unsigned long long *cnt_tile = nullptr;
    unsigned long long *pair_off = nullptr;
};

// ---- launchers (each returns the number of kernels it launched, or -1 on a launch error) ----
// d columns per row starting at column col_lo of vectors that have d_full columns in all
int launch_init_tables(float *U, float *V, uint64_t vocab, uint32_t d, uint32_t ld, uint32_t d_full,
                       uint32_t col_lo, uint64_t seed, cudaStream_t s);

int launch_compact(const int32_t *tokens, uint64_t n, const SampleTables &tab, uint32_t vocab,
                   uint32_t k0, uint32_t k1, uint32_t step_lo, const Scratch &sc, DevState *st,
                   cudaStream_t s);
int launch_windows(uint64_t n, uint32_t window, uint32_t k0, uint32_t k1, uint32_t step_lo,
                   uint32_t il_phase, uint32_t il_stride, const Scratch &sc, DevState *st, cudaStream_t s);
// pair_off[q] = number of pairs of the centres before q; with examples = true, the number of
// centres before q that have at least one context (the example number of the CBOW variant)
// chunks of at most kSmallChunk tokens: counters cleared, sub-sampling, compaction and windows in one launch
constexpr uint64_t kSmallChunk = 8192;
int launch_sample_small(const int32_t *tokens, uint64_t n, const SampleTables &tab, uint32_t vocab, uint32_t k0,
                        uint32_t k1, uint32_t step_lo, uint32_t window, uint32_t il_phase, uint32_t il_stride,
                        const Scratch &sc, DevState *st, cudaStream_t s);
int launch_pair_offsets(uint64_t n, const Scratch &sc, DevState *st, cudaStream_t s, bool examples = false);

// ---- continuous bag of words (w2v_cbow.cu) ----
int launch_cbow_hogwild(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s);
int launch_cbow_snapshot(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s);
int launch_cbow_emit(const StepParams &p, int32_t *centre, int32_t *negs, uint64_t cap, int grid, cudaStream_t s);
int launch_emit_pairs(const StepParams &p, int32_t *centre, int32_t *context, int32_t *negs,
                      uint64_t cap, int grid, cudaStream_t s);
// negs[pair * negatives + k] for every pair of the chunk (needs pair_off); counts the draws
int launch_draw_negatives(const StepParams &p, int32_t *negs, int grid, cudaStream_t s);
// centre[pair], context[pair] and negs[pair * negatives + k] of every pair (needs pair_off); counts the draws
int launch_pair_list(const StepParams &p, int32_t *centre, int32_t *context, int32_t *negs, int grid, cudaStream_t s);

int launch_hogwild(const StepParams &p, uint32_t rows_in_flight, uint32_t blocks_per_sm, int sms,
                   cudaStream_t s);
int launch_snapshot(const StepParams &p, uint32_t rows_in_flight, uint32_t blocks_per_sm, int sms,
                    cudaStream_t s);
// passes 2, 2b and 3 of the snapshot plan alone: G and DU are already filled
int launch_snapshot_apply(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s);
// passes 2b and 3 alone: the fp64 sums of the most-hit rows and the centre sums are applied
int launch_snapshot_tail(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s);
// pass 2b alone (0 launches when no row is summed in fp64)
int launch_apply_hot(const StepParams &p, int sms, cudaStream_t s);
// pass 2 (and the tail) for a column shard: narrow slices put several rows side by side in a warp
int launch_shard_apply(const StepParams &p, uint32_t blocks_per_sm, int sms, cudaStream_t s);

int launch_shard_dots(const StepParams &p, const ShardPeers &peers, int sms, cudaStream_t s);
int launch_shard_coefficients(const float *F, float *G, unsigned long long total, uint32_t n1p, float lr,
                              int sms, cudaStream_t s);
int launch_shard_du(const StepParams &p, int sms, cudaStream_t s);
// one launch; a wait that runs out sets bit 1 of *error
int launch_peer_barrier(const PeerFlags &flags, uint32_t rank, uint32_t epoch, uint32_t timeout_ms, int *error,
                        cudaStream_t s);

int launch_partial_dots(const float *U, const float *V, uint32_t vocab, uint32_t ld,
                        const int32_t *pairs, uint64_t m, uint32_t col_lo, uint32_t col_hi,
                        float *out, DevState *st, int sms, cudaStream_t s);
int launch_copy_rows(float *table, uint32_t vocab, uint32_t d, uint32_t ld, const int64_t *ids, uint64_t m,
                     float *buf, bool to_table, int sms, cudaStream_t s);

// ---- memory-system probe (w2v_probe.cu): `rows` random rows of V in [0, span), returns -2 for d > 512 ----
int launch_probe_rows(float *V, const uint2 *alias, uint32_t vocab, uint32_t d4, uint32_t ld4, uint32_t span,
                      unsigned long long rows, uint32_t access, float *sink, int sms, cudaStream_t s,
                      unsigned long long *rows_done);

// one block per SM pulls `copies` bulk copies of stage_bytes from src[0, span) through a ring of `stages` slots
int launch_probe_mma_ring(const unsigned char *src, unsigned long long stream_stride, uint32_t kps, uint32_t stages, uint32_t tiles,
                          uint32_t span_tiles, int *error, int sms, cudaStream_t s);
int read_probe_mma_ring(long long *cycles, long long *waited);
int launch_probe_bulk_ring(const unsigned char *src, unsigned long long span, uint32_t stage_bytes, uint32_t stages,
                           uint32_t copies, uint32_t producers, int *error, int sms, cudaStream_t s);

// ---- cosine retrieval (w2v_topk.cu) ----
uint32_t topk_splits(uint64_t m, uint64_t n_candidates, int sms, uint32_t block_queries = 0, uint32_t tile_rows = 0, double min_fill = 0.95);
int launch_topk_merge(const float *part_cos, const long long *part_ids, uint64_t m, uint32_t K, uint32_t splits,
                      float *out_cos, long long *out_ids, int sms, cudaStream_t s);
// tensor-core variant (w2v_topk_tc.cu): partial lists only, 128 queries per block, tiles of 256 candidates
size_t topk_tc_qsplit_bytes(uint64_t m, uint32_t d);
int launch_topk_tc(const float *table, uint32_t d, uint32_t ld, uint64_t vocab, const long long *queries, uint64_t m,
                   uint64_t cand_lo, uint64_t cand_hi, uint32_t K, float tau, float *inv_norm,
                   unsigned char *qsplit, unsigned char *ctiles, unsigned int *floor_q, float *part_cos, long long *part_ids,
                   uint32_t splits, int *error, bool screen, bool pairs, int sms, cudaStream_t s);
// inv_norm: 1/|row| of the candidates, an input for the three-MMA kernel (launch_inv_norms); the screening
// variant computes it itself while it packs the candidates.
// The screening variant: how many candidates it handles per launch (a range is cut into chunks of that
// size, each with its own partial lists); bytes of the packed bf16 copy of one chunk.
uint64_t topk_screen_chunk(uint64_t n_candidates, uint32_t d);
size_t topk_screen_ctiles_bytes(uint64_t n_candidates, uint32_t d);
// one block that waits `timeout_ms` on a barrier nobody arrives at and then raises *error (w2v_topk_tc.cu)
int launch_bounded_wait_selftest(uint32_t timeout_ms, int *error, cudaStream_t s);
int launch_inv_norms(const float *table, uint32_t d, uint32_t ld, uint64_t lo, uint64_t count, float *inv_norm,
                     int sms, cudaStream_t s);
// Returns launches made, -1 on a launch error, -2 if the shape does not fit shared memory.
int launch_topk(const float *table, uint32_t d, uint32_t ld, uint64_t vocab, const long long *queries, uint64_t m,
                uint64_t cand_lo, uint64_t cand_hi, uint32_t K, float tau, const float *inv_norm, float *part_cos,
                long long *part_ids, uint32_t splits, float *out_cos, long long *out_ids, int sms, cudaStream_t s);

// ---- host-side table construction (w2v_tables.cpp) ----
// Returns 0, or -1 if a count is zero.  thr_alias is [vocab] pairs, keep_thr [vocab];
// hot_prefix receives the number of leading rows that are drawn as negatives often enough to
// be summed in double precision by the snapshot update.
int build_tables_host(const uint64_t *counts, uint64_t vocab, double subsample_t, uint2 *thr_alias,
                      uint32_t *keep_thr, uint32_t *hot_prefix);

}  // namespace w2v

/*
 * w2v.h -- C ABI of libw2v: the skip-gram negative-sampling (SGNS) minibatch
 * step of "Network-Efficient Distributed Word2vec Training System for Large
 * Vocabularies" (arXiv 1606.08495) on one NVIDIA B200 (sm_100a).
 *
 * The paper spreads one minibatch over parameter-server shards: each shard
 * holds a column slice of every input vector u(w) and output vector v(w),
 * returns partial dot products (Algorithm 1, "dotprod"), the client sums them
 * and forms the coefficients G+ = a(1 - s(F+)), G- = -a s(F-) (Algorithm 3),
 * and the shards apply the linear combinations (Algorithm 2, "adjust").  On
 * one GPU the shards become the lanes of a warp, each owning a column slice,
 * and the two remote calls and the client sum become one kernel.
 *
 * Conventions
 *   - Every function returns a w2v_status (0 = success, negative = error); no
 *     exception crosses this boundary and nothing aborts.  w2v_last_error()
 *     gives a text for the last failure on a handle.
 *   - "device" pointers are CUDA device memory owned by the caller; the
 *     library never frees or reallocates them.  "host" pointers are ordinary
 *     host memory.  The handle owns only its sampling tables and scratch.
 *   - All work is enqueued on the stream given to w2v_create.  Calls that
 *     return values to the host synchronise that stream; the others are
 *     asynchronous.  A handle keeps per-step scratch and counters, so it must
 *     not be used by two host threads at the same time; different handles
 *     are independent.
 *   - Tables are row-major fp32: row w of U (input vectors) or V (output
 *     vectors) is d consecutive floats at offset w*d (w*row_stride for a model
 *     made by w2v_create_strided).  Row index = rank of the word by decreasing
 *     frequency (Section 5.1, the ordering O).
 *   - Token streams are int32 word ids in [0, vocab); -1 ends a sentence;
 *     any other value is skipped as out of vocabulary and reported.  Windows
 *     are taken over the tokens that survive sub-sampling ("dirty" contexts,
 *     footnote to Section 3) and never cross a sentence end or the chunk edge.
 *   - Random choices are a pure function of (seed, step number, token index):
 *     a Philox4x32-10 counter-based generator stands in for the seeded
 *     generator of Algorithms 1 and 2, so that any party regenerates the same
 *     negatives from the same seed, as the paper's shards do.
 *   - Limits: 2 <= vocab < 2^31, d a multiple of 4 with 4 <= d <= 1024,
 *     1 <= window <= 127, 1 <= negatives <= 64, n < 2^31 tokens per call.
 */
#ifndef W2V_H
#define W2V_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct w2v_handle w2v_handle;

typedef enum {
    W2V_OK = 0,
    W2V_ERR_ARG = -1,          /* NULL pointer or value outside the documented limits */
    W2V_ERR_STATE = -2,        /* e.g. a step before w2v_build_alias */
    W2V_ERR_NOMEM = -3,        /* device or host allocation failed */
    W2V_ERR_CUDA = -4,         /* a CUDA runtime call failed; see w2v_last_error */
    W2V_ERR_TOKEN_RANGE = -5,  /* the chunk held ids outside [-1, vocab); they were skipped */
    W2V_ERR_CAPACITY = -6      /* an output array was too small; see the call */
} w2v_status;

enum { W2V_MODE_SNAPSHOT = 0, W2V_MODE_HOGWILD = 1 };
enum { W2V_TABLE_U = 0, W2V_TABLE_V = 1 };

/* Counters of one step (or one w2v_sample_pairs call). */
typedef struct {
    uint64_t tokens;       /* entries in the chunk */
    uint64_t kept;         /* word tokens that survived sub-sampling */
    uint64_t centres;      /* kept tokens with at least one context */
    uint64_t pairs;        /* positive (centre, context) pairs */
    uint64_t neg_draws;    /* alias-table draws, re-draws included */
    uint64_t neg_redraws;  /* draws thrown away because they hit the context word */
    uint64_t oov;          /* ids outside [-1, vocab) */
    uint32_t status;       /* bit 0: out-of-vocabulary ids seen; bit 1: a time-limited wait inside a kernel ran out (W2V_ERR_CUDA) */
    uint32_t reserved;
} w2v_step_stats;

/*
 * Create a model: U ~ uniform[-0.5/d, 0.5/d), V = 0 ("initialized ... as in
 * word2vec", Section 5.1).  U[w][j] = (x - 0.5)/d with x = (r >> 8) 2^-24 and r
 * word j%4 of Philox(key = seed; counter = (w, j/4, 0, 0)).
 *   U, V    device, caller-owned, vocab*d floats each, 16-byte aligned; or both
 *           NULL, in which case the library allocates and owns them.
 *   stream  a cudaStream_t (NULL = the legacy default stream).
 *   out     host; receives the handle.
 * The current CUDA device at the time of the call becomes the handle's device.
 * Asynchronous.  Errors: W2V_ERR_ARG, W2V_ERR_NOMEM, W2V_ERR_CUDA.
 */
int32_t w2v_create(uint64_t vocab, uint32_t d, uint64_t seed, float *U, float *V,
                   void *stream, w2v_handle **out);

/*
 * w2v_create with padded rows: row w of U or V starts at float offset w*row_stride and its
 * first d floats are the vector (the paper fixes only that a vector is an array of d single
 * precision numbers, Section 1; where the rows sit in memory is this library's choice).
 *   row_stride  floats between consecutive rows; a multiple of 4 with d <= row_stride <= 2048.
 *               Recommended: d rounded up to a multiple of 32 floats (320 for d = 300), so that
 *               every row starts on a 128-byte boundary, the granularity at which L2 fetches
 *               and writes back: a gathered row then moves no bytes of its neighbours (measured
 *               on the 60 M x 300 workload: the Hogwild step is 7 % faster than with dense
 *               rows, 6.7 % more memory).  The padding floats are zeroed here and never read
 *               or written afterwards.
 *   U, V        device, caller-owned, vocab*row_stride floats each, 16-byte aligned (128-byte
 *               aligned to get the benefit above); or both NULL (library-owned).
 * Everything else as w2v_create, which is this call with row_stride = d.
 */
int32_t w2v_create_strided(uint64_t vocab, uint32_t d, uint32_t row_stride, uint64_t seed, float *U,
                           float *V, void *stream, w2v_handle **out);

/* Floats between consecutive rows of U and V. */
int32_t w2v_get_row_stride(w2v_handle *h, uint32_t *row_stride);

/* Waits for the handle's stream, frees what the handle owns.  NULL is accepted. */
int32_t w2v_destroy(w2v_handle *h);

/*
 * Build the sampling tables from the vocabulary histogram (Section 5.1: negatives follow a
 * distribution computed from the word counts; Section 3, sub-sampling of frequent words) and
 * upload them.
 *   counts       host, vocab entries, all >= 1 (else W2V_ERR_ARG).
 *   subsample_t  keep probability min(1, sqrt(x) + x), x = t * sum(counts) / count;
 *                t <= 0 keeps every token.
 * Negatives follow count^(3/4) / sum count^(3/4) through a Vose alias table
 * with 32-bit thresholds; weight = sqrt(c) * sqrt(sqrt(c)) in fp64.
 * Synchronises the stream.  May be called again to replace the tables.
 */
int32_t w2v_build_alias(w2v_handle *h, const uint64_t *counts, double subsample_t);

/*
 * Download the tables built by w2v_build_alias (for checking them).
 *   thr, alias, keep_thr  host, vocab entries each; any may be NULL.
 */
int32_t w2v_get_tables(w2v_handle *h, uint32_t *thr, uint32_t *alias, uint32_t *keep_thr);

/*
 * One minibatch step over a chunk of tokens: Eq. (3)-(5), Algorithms 1-3.
 * Sub-sample, compact, draw one window radius b in 1..window per centre, and
 * for every (centre, context) pair draw `negatives` words != context from the
 * alias table; then for every target t of the pair (the context with label 1,
 * the negatives with label 0): F = u(centre).v(t), G = lr (label - s(F)),
 * u(centre) += G v(t), v(t) += G u(centre)  -- summed over the chunk, not averaged.
 *   tokens  device, n int32 entries.
 *   mode    W2V_MODE_SNAPSHOT: every dot and every linear combination uses the
 *           tables as they were at the start of the call and the sums are applied
 *           at the end (Section 5.1: vectors change only when the call ends).
 *           W2V_MODE_HOGWILD: one pass, updates land as they are computed and
 *           later reads may or may not see them (Section 5.1, no locking).
 *   stats   host, may be NULL.  Non-NULL: the call waits for the step and fills
 *           it, and returns W2V_ERR_TOKEN_RANGE if bad ids were skipped.  NULL:
 *           the step is only enqueued and the call does not wait.
 * Adds one to the step number.  Scratch is grown on the first call with a
 * larger n and reused afterwards: no allocation and no waiting in the steady
 * state.  The arrays with one entry per target (snapshot mode's coefficients, the
 * list of negatives of snapshot mode and of Hogwild chunks of 500,000 tokens or
 * more) are sized for the worst case 2 * window * n pairs when that takes at most
 * 1 GiB; only beyond that (wide windows on long chunks) does snapshot mode wait
 * once per step for the pair count and grow them with 25 % head-room, and Hogwild
 * mode draws its negatives inside the update kernel.
 * Errors: W2V_ERR_ARG, W2V_ERR_STATE (no tables), W2V_ERR_NOMEM, W2V_ERR_CUDA
 * (also when status bit 1 reports that a time-limited wait inside a kernel ran out).
 */
int32_t w2v_sgns_step(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window,
                      uint32_t negatives, float lr, uint32_t mode, w2v_step_stats *stats);

/*
 * The same step with the chunk in HOST memory (pinned memory makes the copy
 * asynchronous): copies it to a staging buffer owned by the handle, then
 * behaves exactly as w2v_sgns_step.
 */
int32_t w2v_sgns_step_host(w2v_handle *h, const int32_t *tokens_host, uint64_t n, uint32_t window,
                           uint32_t negatives, float lr, uint32_t mode, w2v_step_stats *stats);

/*
 * The index sets the next step would use (same seed, same step number), without
 * touching the tables or the step number: W_input / W_output of Algorithm 3 and
 * the negatives NS of Algorithms 1 and 2.  Pairs are ordered by centre position,
 * then context position.
 *   centre, context  device, cap int32 each;  negs  device, cap*negatives int32.
 *   n_pairs          host; receives the number of pairs (also when > cap, in
 *                    which case only the first cap are written and the call
 *                    returns W2V_ERR_CAPACITY).
 *   stats            host, may be NULL.
 * Synchronises the stream.
 */
int32_t w2v_sample_pairs(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window,
                         uint32_t negatives, int32_t *centre, int32_t *context, int32_t *negs,
                         uint64_t cap, uint64_t *n_pairs, w2v_step_stats *stats);

/*
 * ---- Continuous bag of words (footnote to Section 5: the paper notes that its design carries
 * over to the CBOW variant and says no more) ------------------------------------------------------
 * One example per kept token q that has at least one context word in its window (window,
 * sub-sampling and dirty contexts exactly as in w2v_sgns_step):
 *   hbar = mean of u(w_k) over the window's context words k (the input table),
 *   targets t: the centre word w_q with label 1 and `negatives` words != w_q with label 0, drawn
 *              from the alias table with the random counter of offset 0 (slot = window),
 *   F = hbar.v(t), G = lr (label - s(F)), v(t) += G hbar, and every context word gets
 *   u(w_k) += (sum_t G v(t)) / |window|   -- lr times the exact gradient of the example's log
 *   likelihood (the open-source word2vec program adds the undivided sum; that is not followed).
 * mode, stats, step number, scratch and errors as for w2v_sgns_step; stats->centres counts the
 * examples and stats->pairs the (centre, context) pairs, i.e. the context rows read.
 * Refused with W2V_ERR_STATE on a column shard.
 */
int32_t w2v_cbow_step(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window,
                      uint32_t negatives, float lr, uint32_t mode, w2v_step_stats *stats);

/* The same with the chunk in HOST memory (see w2v_sgns_step_host). */
int32_t w2v_cbow_step_host(w2v_handle *h, const int32_t *tokens_host, uint64_t n, uint32_t window,
                           uint32_t negatives, float lr, uint32_t mode, w2v_step_stats *stats);

/*
 * The examples the next w2v_cbow_step would use, without touching the tables or the step number:
 * centre word and negatives of example e (examples ordered by centre position).  The context
 * words of the examples are the contexts of w2v_sample_pairs, grouped by centre.
 *   centre  device, cap int32;  negs  device, cap*negatives int32.
 *   n_examples  host; receives the number of examples (also when > cap: W2V_ERR_CAPACITY, the
 *               first cap are written).
 * Synchronises the stream.
 */
int32_t w2v_sample_cbow(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window,
                        uint32_t negatives, int32_t *centre, int32_t *negs, uint64_t cap,
                        uint64_t *n_examples, w2v_step_stats *stats);

/*
 * ---- Column shards: the paper's own partition (Section 5.1, Eq. (6)-(7)) ----------------------
 * Shard s of S holds columns [col_lo, col_hi) of every row of U and V.  One minibatch is
 *   1. every shard: w2v_shard_dots    -- Algorithm 1 ("dotprod") on its slice, for the index
 *                                        sets that every shard regenerates from the same seed;
 *   2. the partial dots are summed over the shards (Algorithm 3, "(F+, F-) <- sum_s");
 *   3. every shard: w2v_shard_adjust  -- G+ = lr (1 - s(F+)), G- = -lr s(F-) (Algorithm 3) and
 *                                        Algorithm 2 ("adjust") on its own columns.
 * Step 2 is either a collective of the caller (w2v_shard_dots adding into one local array, then
 * an all-reduce), or it is done by w2v_shard_dots itself: given the F arrays of all shards
 * (peer-to-peer device pointers), the kernel that computes the partial dots adds them into every
 * one of them, and after a barrier each shard holds the full sums.
 *
 * w2v_create_shard: as w2v_create_strided, for a model that stores only columns
 * [col_lo, col_hi) of vectors that have d_full columns; col_lo and col_hi multiples of 4.
 * Initial values are those the whole model would have in these columns.  U, V: vocab*row_stride
 * floats with row_stride >= col_hi - col_lo.  On the handle of a shard, d means the slice width
 * in every other call (w2v_read_rows returns col_hi - col_lo floats per row; w2v_partial_dots
 * takes columns relative to col_lo), and w2v_sgns_step is refused with W2V_ERR_STATE.
 * All shards must be given the same vocab, d_full, seed, tables, chunks and step numbers.
 */
int32_t w2v_create_shard(uint64_t vocab, uint32_t d_full, uint32_t col_lo, uint32_t col_hi,
                         uint32_t row_stride, uint64_t seed, float *U, float *V, void *stream,
                         w2v_handle **out);

/*
 * Algorithm 1 on this handle's columns for the chunk's index sets (sampled exactly as
 * w2v_sgns_step would).  Target number j = pair*(1+negatives) + t (t = 0 the context word,
 * t >= 1 negative t-1; pairs in the order of w2v_sample_pairs) gets its partial dot product
 * ADDED to F_peers[r][j] for every r < n_peers; with n_peers == 1 it is STORED to F_peers[0][j]
 * (the array then needs no zeroing; entries past the last target are left alone).
 *   tokens   device, n int32.
 *   F_peers  host array of n_peers (1..16) device pointers, each to cap floats that the caller
 *            zeroed before the first shard of this step adds to them; pointers into other
 *            GPUs' memory are allowed when peer access is enabled.
 *   stats    host, may be NULL.
 * Waits once for the pair count.  Returns W2V_ERR_CAPACITY (nothing added) if the chunk has more
 * than cap targets.  Leaves the sampled chunk in the handle for w2v_shard_adjust; any other
 * sampling call or w2v_set_step in between cancels the pending step.
 */
int32_t w2v_shard_dots(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window,
                       uint32_t negatives, float *const *F_peers, uint32_t n_peers, uint64_t cap,
                       w2v_step_stats *stats);

/*
 * Algorithms 3 and 2 for the step begun by w2v_shard_dots: coefficients from the summed dot
 * products, then u(centre) += sum G v(target) and v(target) += G u(centre) on this handle's
 * columns, every vector read as it was at the start of the call.  Adds one to the step number.
 *   F  device, the dot products summed over all shards, indexed as in w2v_shard_dots; every
 *      shard's additions must have completed (the caller's barrier or collective).
 * Asynchronous.  Errors: W2V_ERR_STATE without a pending w2v_shard_dots.
 */
int32_t w2v_shard_adjust(w2v_handle *h, const float *F, float lr);

/*
 * The barrier between w2v_shard_dots and w2v_shard_adjust when the shards add their partial dot
 * products straight into one another's arrays (the sum of Algorithm 3 done over peer pointers):
 * one small kernel on the handle's stream that announces "shard `rank` has finished epoch `epoch`"
 * to every shard and waits until every shard has announced it.  Stream order does the rest: the
 * additions of this shard's w2v_shard_dots precede the announcement, and the w2v_shard_adjust
 * enqueued after the barrier runs only once all announcements have arrived.
 *   flags_peers  host array of n_peers (1..16) device pointers; flags_peers[r] is shard r's array
 *                of n_peers uint32 epoch words (peer-to-peer pointers for r != rank), zeroed once
 *                before the first step and never reset.
 *   rank         which shard this handle is.
 *   epoch        a counter the shards advance together, one per barrier, starting at 1 (compared
 *                modulo 2^32, so it may wrap).
 *   timeout_ms   1..600000.  A shard that never arrives (its process failed before the launch)
 *                must not hang the others' GPUs: when the limit passes the kernel gives up, and
 *                the next w2v_sync on this handle returns W2V_ERR_CUDA once (the step that ran
 *                after the barrier used incomplete sums; the tables are to be restored from a
 *                saved copy).  Nothing traps and the device stays usable.
 * Kernels of different shards wait for one another here, so every shard must be on a GPU of its own
 * (or, for one shard, n_peers == 1).  Asynchronous.
 */
int32_t w2v_peer_barrier(w2v_handle *h, uint32_t *const *flags_peers, uint32_t n_peers, uint32_t rank,
                         uint32_t epoch, uint32_t timeout_ms);

/*
 * Partial dot products of one column slice, the body of Algorithm 1 on shard s:
 * out[i] = sum_{j = col_lo}^{col_hi - 1} U[pairs[2i]][j] * V[pairs[2i+1]][j].
 * Summing the results over any partition of [0, d) gives the full dot products
 * (Algorithm 3, "(F+, F-) <- sum_s").
 *   pairs  device, m*2 int32 (input row, output row), each in [0, vocab).
 *   out    device, m floats.
 * Asynchronous.  Rows out of range leave out[i] = NaN and set status bit 0.
 * Errors: W2V_ERR_ARG unless 0 <= col_lo < col_hi <= d.
 */
int32_t w2v_partial_dots(w2v_handle *h, const int32_t *pairs, uint64_t m, uint32_t col_lo,
                         uint32_t col_hi, float *out);

/*
 * Copy rows out of / into a table (the "get" of the vector export, Section 6.1).
 *   which  W2V_TABLE_U or W2V_TABLE_V.
 *   ids    device, m int64 row numbers; rows outside [0, vocab) are skipped
 *          (read: the output row is left untouched).
 *   out/in device, m*d floats.
 * Asynchronous.
 */
int32_t w2v_read_rows(w2v_handle *h, uint32_t which, const int64_t *ids, uint64_t m, float *out);
int32_t w2v_write_rows(w2v_handle *h, uint32_t which, const int64_t *ids, uint64_t m, const float *in);

/*
 * Retrieval by cosine similarity over the trained vectors (Section 2: top-K by cosine;
 * Section 7.2: K = 30 nearest, kept only above tau = 0.65).
 * For every query row q: among the candidate rows cand_lo <= a < cand_hi, a != q, those with
 * cos(q, a) = x_q.x_a / (|x_q| |x_a|) > tau (a zero row has cosine 0 with everything), and of
 * these the K with the largest cosine, by decreasing cosine, equal cosines by increasing row.
 *   which     W2V_TABLE_U or W2V_TABLE_V (the exported vectors are the input vectors, U).
 *   queries   device, m int64 row numbers; one outside [0, vocab) gets an empty result.
 *   K         1..64;  tau  any float (-2 keeps everything).
 *   out_ids   device, m*K int64, padded with -1;  out_cos  device, m*K floats, padded with 0.
 * Accuracy of the cosines: see w2v_set_retrieval_kernel.  Asynchronous except when scratch
 * (1/|x| per candidate, partial lists) has to grow.  Errors: W2V_ERR_ARG, W2V_ERR_NOMEM,
 * W2V_ERR_CUDA.  Reads the table as it is: call it between steps, not during one.  Scratch grows
 * with m (about 2.6 KB per query at d = 300 for the converted query rows, plus 12 K bytes per query
 * and candidate split for the partial lists): hand large query sets over in batches of some
 * 10^4-10^5.  The default kernel also keeps a bf16 copy of up to 2^22 candidates (at most 2.7 GB).
 */
int32_t w2v_topk_cosine(w2v_handle *h, uint32_t which, const int64_t *queries, uint64_t m,
                        uint64_t cand_lo, uint64_t cand_hi, uint32_t K, float tau, int64_t *out_ids,
                        float *out_cos);

/*
 * Which kernel w2v_topk_cosine runs (the paper has no say in this):
 *   0  fp32 multiply-adds on the CUDA cores: cosines within about 1e-6 of exact;
 *   1  the tensor cores: every value is split into a TF32 head and a TF32 tail and
 *      each product is formed as head*head + head*tail + tail*head in fp32 accumulators that the
 *      hardware updates 3 d/8 times with rounding toward zero: cosines within about
 *      2e-6 + 3 (d/8) 2^-24 of exact (9e-6 at d = 300; 2e-6 typical), at three times the speed.
 *   2  the tensor cores as a screen (the default): queries and unit-length candidates are rounded
 *      to bf16 and one MMA per pair of values gives every cosine to within 8e-3, which decides for
 *      all but a few candidates that they cannot reach the query's current K-th best (or tau); the
 *      few within 8.5e-3 of it are recomputed as fp32 dot products of the two rows, and only those
 *      values are ranked and returned: cosines within about 1e-6 of exact, as with kind 0.  Needs
 *      scratch for the bf16 copy of the candidates (2 d bytes per candidate, at most 2^22
 *      candidates and 2.7 GB at a time: longer ranges are handled in pieces).  Up to 320 columns
 *      the query block stays in shared memory; wider rows stream it beside the candidates.
 *   3  kind 2 on pairs of SMs (`cta_group::2`): two thread blocks of a cluster, each with its own
 *      block of 128 queries and half of every candidate tile, share one stream of candidates; the
 *      same results as kind 2.  Measured on 8192 queries x 3 M candidates of 300 columns: 15.9 ms
 *      against 16.7 ms at tau = 0.65, but 65 ms against 39 ms as a plain top-30 (tau = -2), because
 *      an exact cosine in either block now holds up the accumulators of both; hence not the
 *      default.  Falls back to kind 2 for at most 128 queries or more than 320 columns.
 *   A block of kind 1, 2 or 3 that waits too long on its own pipeline gives up; w2v_sync then
 *   returns W2V_ERR_CUDA.
 */
int32_t w2v_set_retrieval_kernel(w2v_handle *h, uint32_t kind);

/* Step number used by the next step (resume = write the rows back, set the step). */
int32_t w2v_set_step(w2v_handle *h, uint64_t step_id);
int32_t w2v_get_step(w2v_handle *h, uint64_t *step_id);

/*
 * Interleaved minibatch formation (Section 5.1, last paragraph: the input words of a minibatch
 * should be well separated in the corpus, ideally in different sentences).  After this call only
 * the tokens whose index in the chunk is congruent to phase modulo stride act as input (centre)
 * words of w2v_sgns_step, w2v_sample_pairs and w2v_shard_dots; contexts still come from the whole
 * sentence.  Sub-sampling, radii and negatives do not depend on the setting, so the `stride` steps
 * phase = 0..stride-1 over the same chunk WITH THE SAME STEP NUMBER (w2v_set_step before each)
 * use every input word of the chunk exactly once.  stride = 1 (the default) uses them all.
 * Errors: W2V_ERR_ARG unless stride >= 1 and phase < stride.
 */
int32_t w2v_set_interleave(w2v_handle *h, uint32_t phase, uint32_t stride);

/* Device pointers of the two tables (caller's or library-owned). */
int32_t w2v_get_table_ptrs(w2v_handle *h, float **U, float **V);

/* Wait for the handle's stream; returns W2V_ERR_CUDA if a kernel failed. */
int32_t w2v_sync(w2v_handle *h);

/*
 * Timing of the update kernels with CUDA events on the handle's stream.
 * w2v_profile_enable(h, 1) starts recording one event pair around every launch of
 * the step's update kernel(s); w2v_profile_read waits for the stream and returns
 * the summed device time in milliseconds and the number of launches since the
 * last read, then resets both.
 */
int32_t w2v_profile_enable(w2v_handle *h, int32_t on);
int32_t w2v_profile_read(w2v_handle *h, double *kernel_ms, uint64_t *launches);

/* Number of kernels this handle has launched since it was created. */
int32_t w2v_get_launch_count(w2v_handle *h, uint64_t *launches);

/*
 * Exercises the give-up path of the tensor-core retrieval kernels without a fault (no counterpart
 * in the paper: a diagnostic).  Those kernels hand shared-memory stages and accumulators over with
 * barriers, and every wait has a time limit so that a lost hand-over can never hang the GPU; this
 * call enqueues one block that waits, with the same routine, `timeout_ms` (1..2000) on a barrier
 * that nobody arrives at.  The wait runs out, the block raises the handle's error word and returns;
 * the next w2v_sync returns W2V_ERR_CUDA once, and the stream and the device stay usable.
 * Asynchronous.
 */
int32_t w2v_selftest_bounded_wait(w2v_handle *h, uint32_t timeout_ms);

/*
 * Memory-system ceiling for the step's access patterns (no counterpart in the paper: a measuring
 * aid; Section 6 of the paper names the random cache-line rate as what bounds a shard).  Touches
 * `rows` pseudo-random rows of the output table V, drawn uniformly from rows [0, span_rows), with
 * the step kernels' own row layout, 16-byte loads, vector reductions and rows in flight per warp,
 * but without sampling or arithmetic.  Additions add +0.0f: the table keeps its values.
 *   access   W2V_PROBE_GATHER            read each row (what snapshot pass 1 does per target)
 *            W2V_PROBE_GATHER_RED        read each row, then add to it (the Hogwild update)
 *            W2V_PROBE_GATHER_ALIAS      GATHER plus one random 8-byte read of the alias table
 *            W2V_PROBE_GATHER_RED_ALIAS  GATHER_RED plus that read (a negative draw per row)
 *            W2V_PROBE_TOUCH_RED         one word per 64-byte burst, wait, then add (snapshot pass 2)
 *   ms, rows_done  host; receive the kernel's duration (CUDA events on the handle's stream) and
 *            the number of rows it touched (rows rounded up to whole rounds of its launch shape).
 * Synchronises the stream.  Errors: W2V_ERR_ARG (unknown access, span_rows outside 1..vocab,
 * rows outside 1..2^32, d > 512), W2V_ERR_STATE (an ALIAS pattern before w2v_build_alias).
 */
#define W2V_PROBE_GATHER 0u
#define W2V_PROBE_GATHER_RED 1u
#define W2V_PROBE_GATHER_ALIAS 2u
#define W2V_PROBE_GATHER_RED_ALIAS 3u
#define W2V_PROBE_TOUCH_RED 4u
int32_t w2v_probe_rows(w2v_handle *h, uint32_t access, uint64_t span_rows, uint64_t rows, double *ms,
                       uint64_t *rows_done);

/*
 * Second measuring aid (no counterpart in the paper): how fast one SM pulls L2-resident bytes into
 * shared memory through a ring of bulk copies, the way the retrieval kernels stream their
 * candidates.  One block per SM; `producers` lanes issue `cp.async.bulk` copies of stage_bytes
 * from the first 64 MB of V into a ring of `stages` slots as a consumer lane releases them; the
 * consumer only waits and releases.  The retrieval kernels' stage size follows from this figure:
 * a lane hands over about one stage per 250 ns whatever the stage's size.
 *   stage_bytes  a multiple of 16; stage_bytes * stages at most 200 KB;  stages 1..64;  producers 1..4.
 *   bytes_per_sm bytes every block pulls (rounded down to whole stages).
 *   ms, bytes_done  host; the launch's duration and the bytes per block actually copied.
 * Reads V only.  Synchronises the stream.  All waits are bounded; a block that gives up makes
 * the next w2v_sync return W2V_ERR_CUDA.
 */
int32_t w2v_probe_bulk_ring(w2v_handle *h, uint32_t stage_bytes, uint32_t stages, uint32_t producers,
                            uint64_t bytes_per_sm, double *ms, uint64_t *bytes_done);

/*
 * Third measuring aid (no counterpart in the paper): what the feed of the retrieval screen can reach
 * without its epilogue.  One block per SM holds an 80 KB query operand in shared memory; two producer
 * lanes fill a ring of `stages` slots of `kblocks_per_stage` K-blocks (16 KB each, ten per tile of 256
 * candidates) with one bulk copy per slot; one lane issues each tile's 19 bf16 MMAs (128 x 256 x 16) from
 * the slots and commits the slot's release.  Groups of 64 blocks read the same stream of bytes of V
 * (interpreted as bf16: only the timing matters), as the blocks of one candidate split do.
 *   kblocks_per_stage * stages  at most 9 (144 KB of ring);  stages at least 2.
 *   tiles        tiles per block; three streams of tiles * 160 KB must fit into V.
 *   span_tiles   non-zero: a slot holds the next K-blocks whichever tile they belong to; zero: slots do
 *                not span tiles (the last slot of a tile is short), as in the committed kernel.
 *   cycles_per_tile, wait_cycles_per_tile  host; SM cycles per tile of block 0's MMA lane, and the part of
 *                them it spent waiting for data.  The tensor pipe alone needs 19 x 128 = 2432.
 * Reads V only.  Synchronises the stream.  All waits are bounded; a block that gives up makes
 * the next w2v_sync return W2V_ERR_CUDA.
 */
int32_t w2v_probe_mma_ring(w2v_handle *h, uint32_t kblocks_per_stage, uint32_t stages, uint32_t tiles, uint32_t span_tiles,
                           double *cycles_per_tile, double *wait_cycles_per_tile);

/*
 * Launch shape of the update kernels: rows in flight per warp (1..8; 0 = default)
 * and resident thread blocks per SM (0 = as many as fit).  Results do not depend
 * on it in snapshot mode.
 */
int32_t w2v_set_tuning(w2v_handle *h, uint32_t rows_in_flight, uint32_t blocks_per_sm);

/*
 * w2v_sample_pairs for callers that must not allocate device memory.  (The paper has no
 * counterpart to this call; it exists for the sake of the library's users.)
 *
 * Who needs it: code that runs when the rest of the GPU's memory already belongs to someone
 * else (a training framework's caching allocator, a serving engine's KV cache), code on a
 * latency-critical path where the implicit synchronisation of an allocation is unwelcome, and
 * hosts whose policy is "no allocation after start-up".  w2v_sample_pairs grows scratch inside
 * the handle on first use; this variant never calls cudaMalloc, cudaFree or any other
 * allocating routine.  Its scratch is one fixed array of just under 2 MiB inside the library
 * image, present on every GPU that loads the library until the process exits.
 *
 * Same arguments, same results and the same return codes as w2v_sample_pairs, except:
 *   - n may be at most 65536 tokens; a larger chunk is refused with W2V_ERR_CAPACITY
 *     ("serves at most 65536 tokens per call") before anything is launched.
 *   - The first call on each GPU looks up the device address of the fixed array.  Make that
 *     first call during set-up, before any CUDA stream capture begins, and from one host
 *     thread: two first calls on the same GPU at the same moment would both store the (same)
 *     address into the library's per-GPU cache without synchronisation.
 *   - All handles and all calls on one GPU share the one array, and it keeps whatever the
 *     previous call left in it (this call clears the counters it needs at zero).  Two calls
 *     that overlap on the GPU -- from different streams or threads -- race on it; issue
 *     them one after the other.  The call returns only after its own work has finished.
 */
int32_t w2v_sample_pairs_noalloc(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window,
                                 uint32_t negatives, int32_t *centre, int32_t *context, int32_t *negs,
                                 uint64_t cap, uint64_t *n_pairs, w2v_step_stats *stats);

/* Text of the last error on this handle (never NULL; h == NULL gives a generic text). */
const char *w2v_last_error(w2v_handle *h);

#ifdef __cplusplus
}
#endif
#endif /* W2V_H */

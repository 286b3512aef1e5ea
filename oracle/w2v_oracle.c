/*
 * w2v_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-threaded CPU statement of the skip-gram
 * negative-sampling (SGNS) minibatch step of "Network-Efficient Distributed
 * Word2vec Training System for Large Vocabularies" (arXiv 1606.08495).
 * It exists so that the CUDA library can be checked against something that a
 * reader can compare with the paper by eye.  It shares no code, header, table
 * or constant generator with the CUDA library and must never be called from
 * the product path: only the tests, the smoke check and the benchmark's
 * cpu-baseline / reference arm may load it.
 *
 * Storage is fp32 (Section 1: vectors are single precision arrays); every
 * dot product, sigmoid, coefficient and linear combination is evaluated in
 * fp64 and rounded to fp32 once, when a row is written back.
 *
 * What each part follows:
 *   philox4x32_10      the published Philox4x32-10 counter-based generator
 *                      (Salmon et al., SC'11); stands in for the seeded random
 *                      number generator of Algorithms 1 and 2,
 *                      so that the same seed regenerates the same negatives.
 *   orc_init_row       initial values as in the word2vec program
 *                      (Section 5.1): input rows uniform in [-0.5/d, 0.5/d),
 *                      output rows zero.
 *   build_alias        negative-example distribution computed from the
 *                      word counts (Section 5.1, dotprod item):
 *                      unigram^(3/4), sampled through a Vose alias table.
 *   build_keep         sub-sampling of frequent words (Section 3, last lines).
 *   sample_chunk       Eq. (1)/(3) index sets: dirty contexts (footnote to
 *                      Section 3), random window radius b, N negatives != w_O
 *                      (Algorithm 1, the array NS of negatives).
 *   orc_step mode 0    Algorithm 1 + Algorithm 3 (aggregation, G+ / G-) +
 *                      Algorithm 2 literally: all reads see start-of-call
 *                      values, deltas are applied at the end (Section 5.1:
 *                      vectors change only when the call ends).
 *   orc_step mode 1    the sequential limit of the lock-free operation of
 *                      Section 5.1: targets one after another, every read sees
 *                      every earlier write.
 *   orc_set_interleave interleaved minibatch formation (Section 5.1, last
 *                      paragraph): the input words of one call are a stride apart.
 *   orc_cbow_*         the continuous-bag-of-words variant (footnote to
 *                      Section 5, which only notes that the design carries
 *                      over to CBOW): the mean of the
 *                      context words' input vectors predicts the centre word;
 *                      same index sets, same two modes, exact gradient.
 *   orc_topk_cosine    retrieval by cosine similarity (Section 2: top-K by
 *                      cosine; Section 7.2: K nearest, kept only above a
 *                      threshold tau): brute force.
 *   orc_partial_dots   u_s(w_I) v_s(w_O)^T of Algorithm 1 for one column slice.
 *   orc_loss           minus Eq. (1) restricted to a chunk, per positive pair.
 *
 * Parity pins (tests/test_oracle_*.py): published known-answer vectors of
 * Philox4x32-10; exact alias-table distribution against brute-force
 * c^0.75 / sum c^0.75; hand-computed 3-word examples; Eq. (4) against central
 * finite differences of Eq. (3); first-step closed form with V = 0; the
 * slice-sum identity of Algorithm 3 line "(F+,F-) <- sum_s"; hand-enumerated
 * windows; for CBOW: finite differences of its objective, the one-context case
 * that reduces to a skip-gram pair, and the first-step closed form; for the
 * retrieval: vectors with known angles, scale invariance, a full sort by numpy.
 * No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (published algorithm; 10 rounds, key bumped between). */
/* ------------------------------------------------------------------ */
static void philox4x32_10(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1,
                          uint32_t c2, uint32_t c3, uint32_t out[4])
{
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = M0 * (uint64_t)c0;
        uint64_t p1 = M1 * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

void orc_philox(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1,
                uint32_t c2, uint32_t c3, uint32_t *out)
{
    philox4x32_10(k0, k1, c0, c1, c2, c3, out);
}

/* Counter layout.  c0 = position (token index in the chunk, or row for init),
 * c1 = low word of the step number, c2 = purpose | slot << 8,
 * c3 = k | attempt << 16.  The high word of the step is folded into the key. */
enum { PUR_INIT = 0, PUR_SUBSAMPLE = 1, PUR_RADIUS = 2, PUR_NEGATIVE = 3 };

/* ------------------------------------------------------------------ */
/* A small growable map  int64 key -> uint32 value  (open addressing).  */
/* ------------------------------------------------------------------ */
typedef struct {
    int64_t *keys;
    uint32_t *vals;
    uint64_t cap; /* power of two */
    uint64_t count;
} idmap;

static void idmap_init(idmap *m, uint64_t cap)
{
    m->cap = 1024;
    while (m->cap < cap) m->cap <<= 1;
    m->keys = (int64_t *)malloc(m->cap * sizeof(int64_t));
    m->vals = (uint32_t *)malloc(m->cap * sizeof(uint32_t));
    for (uint64_t i = 0; i < m->cap; ++i) m->keys[i] = -1;
    m->count = 0;
}
static void idmap_free(idmap *m)
{
    free(m->keys); free(m->vals);
    m->keys = NULL; m->vals = NULL; m->cap = 0; m->count = 0;
}
static uint64_t idmap_slot(const idmap *m, int64_t key)
{
    uint64_t h = (uint64_t)key * 0x9E3779B97F4A7C15ull;
    h ^= h >> 29;
    return h & (m->cap - 1);
}
/* returns 1 and *val when present */
static int idmap_get(const idmap *m, int64_t key, uint32_t *val)
{
    uint64_t s = idmap_slot(m, key);
    while (m->keys[s] != -1) {
        if (m->keys[s] == key) { *val = m->vals[s]; return 1; }
        s = (s + 1) & (m->cap - 1);
    }
    return 0;
}
static void idmap_put(idmap *m, int64_t key, uint32_t val);
static void idmap_grow(idmap *m)
{
    idmap big;
    idmap_init(&big, m->cap * 2);
    for (uint64_t i = 0; i < m->cap; ++i)
        if (m->keys[i] != -1) idmap_put(&big, m->keys[i], m->vals[i]);
    idmap_free(m);
    *m = big;
}
static void idmap_put(idmap *m, int64_t key, uint32_t val)
{
    if ((m->count + 1) * 2 > m->cap) idmap_grow(m);
    uint64_t s = idmap_slot(m, key);
    while (m->keys[s] != -1 && m->keys[s] != key) s = (s + 1) & (m->cap - 1);
    if (m->keys[s] == -1) m->count++;
    m->keys[s] = key;
    m->vals[s] = val;
}

/* ------------------------------------------------------------------ */
/* Row store: fp32 rows of the input table U and the output table V.   */
/* Dense: one array.  Sparse: rows come into being, with their initial  */
/* value, the first time they are touched (for vocabularies whose dense */
/* tables do not fit in host memory).                                    */
/* ------------------------------------------------------------------ */
#define CHUNK_ROWS 16384u

typedef struct {
    int sparse;
    int is_input;      /* 1: U (random init), 0: V (zero init) */
    uint64_t vocab;
    uint32_t d;
    float *dense;
    idmap map;         /* sparse: row -> slot */
    float **chunks;
    uint32_t n_chunks, cap_chunks;
    uint64_t n_rows;
} rowstore;

typedef struct orc {
    uint64_t vocab;
    uint32_t d;
    uint64_t seed;
    uint64_t step_id;
    uint32_t il_phase, il_stride;   /* interleaved minibatches: centres with index % stride == phase */
    rowstore U, V;
    int have_tables;
    uint32_t *thr;     /* alias acceptance thresholds (units of 2^-32) */
    uint32_t *alias;
    uint32_t *keep_thr;
    /* last sampled chunk */
    int32_t *ctok; uint32_t *cidx; uint32_t *csent; uint64_t cap_kept;
    /* counters of the last sampling pass */
    uint64_t st_tokens, st_kept, st_centres, st_pairs, st_draws, st_redraws, st_oov;
} orc;

static void init_row_values(const orc *h, uint64_t row, float *out)
{
    /* u[row][j] = (x - 0.5) / d with x = top 24 bits of a Philox word * 2^-24;
     * one Philox call yields four consecutive columns. */
    uint32_t k0 = (uint32_t)h->seed, k1 = (uint32_t)(h->seed >> 32);
    for (uint32_t j = 0; j < h->d; j += 4) {
        uint32_t r[4];
        philox4x32_10(k0, k1, (uint32_t)row, j / 4, PUR_INIT, 0, r);
        for (uint32_t e = 0; e < 4 && j + e < h->d; ++e) {
            float x = (float)(r[e] >> 8) * (1.0f / 16777216.0f);
            out[j + e] = (x - 0.5f) / (float)h->d;
        }
    }
}

static void rs_init(rowstore *rs, const orc *h, int is_input, int sparse)
{
    memset(rs, 0, sizeof(*rs));
    rs->sparse = sparse; rs->is_input = is_input;
    rs->vocab = h->vocab; rs->d = h->d;
    if (!sparse) {
        rs->dense = (float *)calloc((size_t)h->vocab * h->d, sizeof(float));
        if (is_input)
            for (uint64_t w = 0; w < h->vocab; ++w)
                init_row_values(h, w, rs->dense + (size_t)w * h->d);
    } else {
        idmap_init(&rs->map, 1u << 16);
        rs->cap_chunks = 64;
        rs->chunks = (float **)calloc(rs->cap_chunks, sizeof(float *));
    }
}
static void rs_free(rowstore *rs)
{
    if (!rs->sparse) { free(rs->dense); return; }
    for (uint32_t i = 0; i < rs->n_chunks; ++i) free(rs->chunks[i]);
    free(rs->chunks);
    idmap_free(&rs->map);
}
static float *rs_row(rowstore *rs, const orc *h, uint64_t row)
{
    if (!rs->sparse) return rs->dense + (size_t)row * rs->d;
    uint32_t slot;
    if (!idmap_get(&rs->map, (int64_t)row, &slot)) {
        slot = (uint32_t)rs->n_rows++;
        uint32_t ch = slot / CHUNK_ROWS;
        if (ch >= rs->n_chunks) {
            if (ch >= rs->cap_chunks) {
                rs->cap_chunks *= 2;
                rs->chunks = (float **)realloc(rs->chunks, rs->cap_chunks * sizeof(float *));
            }
            rs->chunks[ch] = (float *)calloc((size_t)CHUNK_ROWS * rs->d, sizeof(float));
            rs->n_chunks = ch + 1;
        }
        idmap_put(&rs->map, (int64_t)row, slot);
        float *p = rs->chunks[ch] + (size_t)(slot % CHUNK_ROWS) * rs->d;
        if (rs->is_input) init_row_values(h, row, p);
        return p;
    }
    return rs->chunks[slot / CHUNK_ROWS] + (size_t)(slot % CHUNK_ROWS) * rs->d;
}

/* ------------------------------------------------------------------ */
/* Handle                                                               */
/* ------------------------------------------------------------------ */
orc *orc_create(uint64_t vocab, uint32_t d, uint64_t seed, int sparse)
{
    if (vocab < 2 || vocab >= (1ull << 31) || d == 0) return NULL;
    orc *h = (orc *)calloc(1, sizeof(orc));
    h->vocab = vocab; h->d = d; h->seed = seed; h->step_id = 0;
    rs_init(&h->U, h, 1, sparse);
    rs_init(&h->V, h, 0, sparse);
    return h;
}
void orc_destroy(orc *h)
{
    if (!h) return;
    rs_free(&h->U); rs_free(&h->V);
    free(h->thr); free(h->alias); free(h->keep_thr);
    free(h->ctok); free(h->cidx); free(h->csent);
    free(h);
}
void orc_set_step(orc *h, uint64_t s) { h->step_id = s; }
/* Interleaved minibatch formation (Section 5.1, last paragraph): of the chunk's kept tokens only
 * those whose index in the chunk is congruent to phase modulo stride act as input (centre) words;
 * their contexts are still taken from the whole sentence.  The `stride` calls phase = 0..stride-1
 * with the same step number cover every input word of the chunk exactly once, and the input words
 * of one call are at least `stride` tokens apart. */
int orc_set_interleave(orc *h, uint32_t phase, uint32_t stride)
{
    if (stride < 1 || phase >= stride) return -1;
    h->il_phase = phase; h->il_stride = stride;
    return 0;
}
uint64_t orc_get_step(const orc *h) { return h->step_id; }

void orc_init_row(const orc *h, uint64_t row, float *out) { init_row_values(h, row, out); }

void orc_read_rows(orc *h, uint32_t which, const int64_t *ids, uint64_t m, float *out)
{
    rowstore *rs = which ? &h->V : &h->U;
    for (uint64_t i = 0; i < m; ++i)
        memcpy(out + (size_t)i * h->d, rs_row(rs, h, (uint64_t)ids[i]), h->d * sizeof(float));
}
void orc_write_rows(orc *h, uint32_t which, const int64_t *ids, uint64_t m, const float *in)
{
    rowstore *rs = which ? &h->V : &h->U;
    for (uint64_t i = 0; i < m; ++i)
        memcpy(rs_row(rs, h, (uint64_t)ids[i]), in + (size_t)i * h->d, h->d * sizeof(float));
}

/* ------------------------------------------------------------------ */
/* Sampling tables                                                      */
/* ------------------------------------------------------------------ */
/* Negative distribution p_i = c_i^(3/4) / sum_j c_j^(3/4), as a Vose alias
 * table with 32-bit acceptance thresholds.  The weight is formed as
 * sqrt(c) * sqrt(sqrt(c)) (three correctly rounded operations) so that an
 * independent implementation reproduces every bit. */
static int build_alias(orc *h, const uint64_t *counts)
{
    uint64_t V = h->vocab;
    double *q = (double *)malloc(V * sizeof(double));
    uint32_t *small = (uint32_t *)malloc(V * sizeof(uint32_t));
    uint32_t *large = (uint32_t *)malloc(V * sizeof(uint32_t));
    uint64_t ns = 0, nl = 0;
    double wsum = 0.0;
    for (uint64_t i = 0; i < V; ++i) {
        if (counts[i] == 0) { free(q); free(small); free(large); return -1; }
        double c = (double)counts[i];
        double r = sqrt(c);
        q[i] = r * sqrt(r);
        wsum += q[i];
    }
    for (uint64_t i = 0; i < V; ++i) {
        q[i] = (q[i] * (double)V) / wsum;
        if (q[i] < 1.0) small[ns++] = (uint32_t)i; else large[nl++] = (uint32_t)i;
    }
    for (uint64_t i = 0; i < V; ++i) { h->thr[i] = 0xFFFFFFFFu; h->alias[i] = (uint32_t)i; }
    while (ns > 0 && nl > 0) {
        uint32_t s = small[--ns];
        uint32_t l = large[--nl];
        double scaled = floor(q[s] * 4294967296.0);
        h->thr[s] = scaled >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)scaled;
        h->alias[s] = l;
        q[l] = (q[l] + q[s]) - 1.0;
        if (q[l] < 1.0) small[ns++] = l; else large[nl++] = l;
    }
    /* whatever is left on either stack keeps thr = 2^32-1, alias = itself */
    free(q); free(small); free(large);
    return 0;
}

/* Keep probability of the open-source word2vec program, which the paper
 * defers to: p = sqrt(x) + x with x = t * total / c_w, capped at 1. */
static void build_keep(orc *h, const uint64_t *counts, double t)
{
    uint64_t total = 0;
    for (uint64_t i = 0; i < h->vocab; ++i) total += counts[i];
    for (uint64_t i = 0; i < h->vocab; ++i) {
        if (!(t > 0.0)) { h->keep_thr[i] = 0xFFFFFFFFu; continue; }
        double x = (t * (double)total) / (double)counts[i];
        double p = sqrt(x) + x;
        if (p >= 1.0) { h->keep_thr[i] = 0xFFFFFFFFu; continue; }
        h->keep_thr[i] = (uint32_t)floor(p * 4294967296.0);
    }
}

int orc_build_tables(orc *h, const uint64_t *counts, double subsample_t)
{
    if (!h->thr) {
        h->thr = (uint32_t *)malloc(h->vocab * sizeof(uint32_t));
        h->alias = (uint32_t *)malloc(h->vocab * sizeof(uint32_t));
        h->keep_thr = (uint32_t *)malloc(h->vocab * sizeof(uint32_t));
    }
    if (build_alias(h, counts) != 0) return -1;
    build_keep(h, counts, subsample_t);
    h->have_tables = 1;
    return 0;
}
int orc_get_tables(const orc *h, uint32_t *thr, uint32_t *alias, uint32_t *keep_thr)
{
    if (!h->have_tables) return -1;
    memcpy(thr, h->thr, h->vocab * sizeof(uint32_t));
    memcpy(alias, h->alias, h->vocab * sizeof(uint32_t));
    memcpy(keep_thr, h->keep_thr, h->vocab * sizeof(uint32_t));
    return 0;
}

/* One draw from the alias table: 64 random bits choose the bucket by a
 * multiply-high with V, 32 more bits accept it or take its alias. */
static uint32_t alias_draw(const orc *h, const uint32_t r[4])
{
    unsigned __int128 wide = (unsigned __int128)(((uint64_t)r[0] << 32) | r[1]) * (unsigned __int128)h->vocab;
    uint32_t bucket = (uint32_t)(uint64_t)(wide >> 64);
    return r[2] < h->thr[bucket] ? bucket : h->alias[bucket];
}
uint32_t orc_alias_draw(const orc *h, uint32_t r0, uint32_t r1, uint32_t r2)
{
    uint32_t r[4] = { r0, r1, r2, 0 };
    return alias_draw(h, r);
}

/* ------------------------------------------------------------------ */
/* Index sets of Eq. (3) for one chunk of tokens                        */
/* ------------------------------------------------------------------ */
typedef void (*pair_fn)(void *ctx, uint64_t pair_index, int32_t centre, int32_t context,
                        const int32_t *negs, uint32_t N);

/* tokens: ids in [0, vocab); -1 ends a sentence; anything else is out of
 * vocabulary and is skipped.  Windows are taken over the kept tokens only
 * ("dirty" contexts) and never cross a sentence end or the chunk edge.
 * Pairs come out ordered by centre position, then context position. */
static void sample_chunk(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N,
                         uint64_t step_id, pair_fn fn, void *ctx)
{
    uint32_t k0 = (uint32_t)h->seed;
    uint32_t k1 = (uint32_t)(h->seed >> 32) ^ (uint32_t)(step_id >> 32);
    uint32_t step_lo = (uint32_t)step_id;
    if (h->cap_kept < n + 1) {
        free(h->ctok); free(h->cidx); free(h->csent);
        h->cap_kept = n + 1;
        h->ctok = (int32_t *)malloc(h->cap_kept * sizeof(int32_t));
        h->cidx = (uint32_t *)malloc(h->cap_kept * sizeof(uint32_t));
        h->csent = (uint32_t *)malloc(h->cap_kept * sizeof(uint32_t));
    }
    h->st_tokens = n; h->st_kept = h->st_centres = h->st_pairs = 0;
    h->st_draws = h->st_redraws = h->st_oov = 0;

    /* sub-sampling and compaction */
    uint64_t nk = 0;
    uint32_t sent = 0;
    for (uint64_t i = 0; i < n; ++i) {
        int32_t w = tokens[i];
        if (w == -1) { sent++; continue; }
        if (w < 0 || (uint64_t)w >= h->vocab) { h->st_oov++; continue; }
        uint32_t thr = h->keep_thr[w];
        if (thr != 0xFFFFFFFFu) {
            uint32_t r[4];
            philox4x32_10(k0, k1, (uint32_t)i, step_lo, PUR_SUBSAMPLE, 0, r);
            if (!(r[0] < thr)) continue;
        }
        h->ctok[nk] = w; h->cidx[nk] = (uint32_t)i; h->csent[nk] = sent;
        nk++;
    }
    h->st_kept = nk;

    int32_t negs[64];
    uint64_t pair_index = 0;
    for (uint64_t q = 0; q < nk; ++q) {
        uint32_t r[4];
        if (h->il_stride > 1 && h->cidx[q] % h->il_stride != h->il_phase) continue;
        philox4x32_10(k0, k1, h->cidx[q], step_lo, PUR_RADIUS, 0, r);
        int64_t b = 1 + (int64_t)(((uint64_t)r[0] * (uint64_t)W) >> 32);
        int had = 0;
        for (int64_t p = (int64_t)q - b; p <= (int64_t)q + b; ++p) {
            if (p == (int64_t)q || p < 0 || p >= (int64_t)nk) continue;
            if (h->csent[p] != h->csent[q]) continue;
            int32_t wO = h->ctok[p];
            uint32_t slot = (uint32_t)(p - (int64_t)q + (int64_t)W);
            for (uint32_t k = 0; k < N; ++k) {
                uint32_t cand = 0;
                int found = 0;
                for (uint32_t a = 0; a < 16 && !found; ++a) {
                    philox4x32_10(k0, k1, h->cidx[q], step_lo, PUR_NEGATIVE | (slot << 8),
                                  k | (a << 16), r);
                    cand = alias_draw(h, r);
                    h->st_draws++;
                    if (cand != (uint32_t)wO) found = 1; else h->st_redraws++;
                }
                if (!found) cand = (uint32_t)(((uint64_t)wO + 1) % h->vocab);
                negs[k] = (int32_t)cand;
            }
            fn(ctx, pair_index++, h->ctok[q], wO, negs, N);
            had = 1;
        }
        if (had) h->st_centres++;
    }
    h->st_pairs = pair_index;
}

void orc_get_stats(const orc *h, uint64_t *out7)
{
    out7[0] = h->st_tokens; out7[1] = h->st_kept; out7[2] = h->st_centres; out7[3] = h->st_pairs;
    out7[4] = h->st_draws; out7[5] = h->st_redraws; out7[6] = h->st_oov;
}

/* ---- materialise the pair list ------------------------------------ */
typedef struct { int32_t *centre, *context, *negs; uint64_t cap; } pairsink;
static void sink_pair(void *ctx, uint64_t pi, int32_t c, int32_t o, const int32_t *negs, uint32_t N)
{
    pairsink *s = (pairsink *)ctx;
    if (pi >= s->cap) return;
    s->centre[pi] = c; s->context[pi] = o;
    for (uint32_t k = 0; k < N; ++k) s->negs[pi * N + k] = negs[k];
}
int orc_sample_pairs(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N,
                     int32_t *centre, int32_t *context, int32_t *negs, uint64_t cap,
                     uint64_t *n_pairs)
{
    if (!h->have_tables || W < 1 || W > 127 || N < 1 || N > 64) return -1;
    pairsink s = { centre, context, negs, cap };
    sample_chunk(h, tokens, n, W, N, h->step_id, sink_pair, &s);
    *n_pairs = h->st_pairs;
    return 0;
}

/* ------------------------------------------------------------------ */
/* The step                                                             */
/* ------------------------------------------------------------------ */
static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

static double dot_rows(const float *a, const float *b, uint32_t lo, uint32_t hi)
{
    double s = 0.0;
    for (uint32_t j = lo; j < hi; ++j) s += (double)a[j] * (double)b[j];
    return s;
}

/* -- mode 1: one target after another, each seeing all earlier writes -- */
typedef struct { orc *h; double lr; double *e; } seqctx;
static void seq_pair(void *ctx, uint64_t pi, int32_t c, int32_t o, const int32_t *negs, uint32_t N)
{
    (void)pi;
    seqctx *s = (seqctx *)ctx;
    orc *h = s->h;
    uint32_t d = h->d;
    float *u = rs_row(&h->U, h, (uint64_t)c);
    for (uint32_t j = 0; j < d; ++j) s->e[j] = 0.0;
    for (uint32_t k = 0; k <= N; ++k) {
        int32_t t = k == 0 ? o : negs[k - 1];
        double label = k == 0 ? 1.0 : 0.0;
        float *v = rs_row(&h->V, h, (uint64_t)t);
        double f = dot_rows(u, v, 0, d);
        double g = s->lr * (label - sigmoid(f));
        for (uint32_t j = 0; j < d; ++j) s->e[j] += g * (double)v[j];
        for (uint32_t j = 0; j < d; ++j) v[j] = (float)((double)v[j] + g * (double)u[j]);
    }
    for (uint32_t j = 0; j < d; ++j) u[j] = (float)((double)u[j] + s->e[j]);
}

/* -- mode 0: dotprod, coefficients, adjust with deferred application -- */
typedef struct {
    orc *h; double lr;
    idmap du_map, dv_map;      /* row -> index into the delta pools */
    double *du, *dv; uint64_t ndu, ndv, capdu, capdv;
} snapctx;
static double *delta_row(snapctx *s, int is_u, int64_t row)
{
    idmap *m = is_u ? &s->du_map : &s->dv_map;
    double **pool = is_u ? &s->du : &s->dv;
    uint64_t *cnt = is_u ? &s->ndu : &s->ndv, *cap = is_u ? &s->capdu : &s->capdv;
    uint32_t d = s->h->d, idx;
    if (!idmap_get(m, row, &idx)) {
        if (*cnt == *cap) {
            *cap = *cap ? *cap * 2 : 4096;
            *pool = (double *)realloc(*pool, (size_t)*cap * d * sizeof(double));
        }
        idx = (uint32_t)(*cnt)++;
        memset(*pool + (size_t)idx * d, 0, d * sizeof(double));
        idmap_put(m, row, idx);
    }
    return *pool + (size_t)idx * d;
}
static void snap_pair(void *ctx, uint64_t pi, int32_t c, int32_t o, const int32_t *negs, uint32_t N)
{
    (void)pi;
    snapctx *s = (snapctx *)ctx;
    orc *h = s->h;
    uint32_t d = h->d;
    const float *u = rs_row(&h->U, h, (uint64_t)c);   /* untouched until the end of the step */
    for (uint32_t k = 0; k <= N; ++k) {
        int32_t t = k == 0 ? o : negs[k - 1];
        const float *v = rs_row(&h->V, h, (uint64_t)t);
        double f = dot_rows(u, v, 0, d);                                  /* Algorithm 1 */
        double g = k == 0 ? s->lr * (1.0 - sigmoid(f)) : -s->lr * sigmoid(f); /* Algorithm 3 */
        double *dv = delta_row(s, 0, t);                                  /* Algorithm 2 */
        for (uint32_t j = 0; j < d; ++j) dv[j] += g * (double)u[j];
        double *du = delta_row(s, 1, c);
        for (uint32_t j = 0; j < d; ++j) du[j] += g * (double)v[j];
    }
}
static void snap_apply(snapctx *s, int is_u)
{
    orc *h = s->h;
    idmap *m = is_u ? &s->du_map : &s->dv_map;
    double *pool = is_u ? s->du : s->dv;
    rowstore *rs = is_u ? &h->U : &h->V;
    for (uint64_t i = 0; i < m->cap; ++i) {
        if (m->keys[i] == -1) continue;
        float *x = rs_row(rs, h, (uint64_t)m->keys[i]);
        const double *dx = pool + (size_t)m->vals[i] * h->d;
        for (uint32_t j = 0; j < h->d; ++j) x[j] = (float)((double)x[j] + dx[j]);
    }
}

int orc_step(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N, double lr, uint32_t mode)
{
    if (!h->have_tables || W < 1 || W > 127 || N < 1 || N > 64 || mode > 1) return -1;
    if (mode == 1) {
        seqctx s = { h, lr, (double *)malloc(h->d * sizeof(double)) };
        sample_chunk(h, tokens, n, W, N, h->step_id, seq_pair, &s);
        free(s.e);
    } else {
        snapctx s;
        memset(&s, 0, sizeof(s));
        s.h = h; s.lr = lr;
        idmap_init(&s.du_map, 4096); idmap_init(&s.dv_map, 4096);
        sample_chunk(h, tokens, n, W, N, h->step_id, snap_pair, &s);
        snap_apply(&s, 1);
        snap_apply(&s, 0);
        idmap_free(&s.du_map); idmap_free(&s.dv_map);
        free(s.du); free(s.dv);
    }
    h->step_id++;
    return 0;
}

/* Apply one step to an explicit list of (centre, context, negatives): the
 * same arithmetic as orc_step with the sampling taken out, for hand examples. */
int orc_step_pairs(orc *h, const int32_t *centre, const int32_t *context, const int32_t *negs,
                   uint64_t P, uint32_t N, double lr, uint32_t mode)
{
    if (mode > 1 || N > 64) return -1;
    if (mode == 1) {
        seqctx s = { h, lr, (double *)malloc(h->d * sizeof(double)) };
        for (uint64_t p = 0; p < P; ++p) seq_pair(&s, p, centre[p], context[p], negs + p * N, N);
        free(s.e);
    } else {
        snapctx s;
        memset(&s, 0, sizeof(s));
        s.h = h; s.lr = lr;
        idmap_init(&s.du_map, 4096); idmap_init(&s.dv_map, 4096);
        for (uint64_t p = 0; p < P; ++p) snap_pair(&s, p, centre[p], context[p], negs + p * N, N);
        snap_apply(&s, 1);
        snap_apply(&s, 0);
        idmap_free(&s.du_map); idmap_free(&s.dv_map);
        free(s.du); free(s.dv);
    }
    return 0;
}

/* -- partial dot products of one column slice (Algorithm 1 on shard s) -- */
int orc_partial_dots(orc *h, const int32_t *pairs, uint64_t m, uint32_t col_lo, uint32_t col_hi, double *out)
{
    if (!(col_lo < col_hi && col_hi <= h->d)) return -1;
    for (uint64_t i = 0; i < m; ++i) {
        const float *u = rs_row(&h->U, h, (uint64_t)pairs[2 * i]);
        const float *v = rs_row(&h->V, h, (uint64_t)pairs[2 * i + 1]);
        out[i] = dot_rows(u, v, col_lo, col_hi);
    }
    return 0;
}

/* -- minus the log likelihood of Eq. (1) over a chunk, per positive pair -- */
static double log_sigmoid(double x)
{
    return x >= 0.0 ? -log1p(exp(-x)) : x - log1p(exp(x));
}
typedef struct { orc *h; double sum; } lossctx;
static void loss_pair(void *ctx, uint64_t pi, int32_t c, int32_t o, const int32_t *negs, uint32_t N)
{
    (void)pi;
    lossctx *s = (lossctx *)ctx;
    orc *h = s->h;
    const float *u = rs_row(&h->U, h, (uint64_t)c);
    s->sum += log_sigmoid(dot_rows(u, rs_row(&h->V, h, (uint64_t)o), 0, h->d));
    for (uint32_t k = 0; k < N; ++k)
        s->sum += log_sigmoid(-dot_rows(u, rs_row(&h->V, h, (uint64_t)negs[k]), 0, h->d));
}
int orc_loss(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N, uint64_t step_id,
             double *loss_sum, uint64_t *n_pairs)
{
    if (!h->have_tables || W < 1 || W > 127 || N < 1 || N > 64) return -1;
    lossctx s = { h, 0.0 };
    sample_chunk(h, tokens, n, W, N, step_id, loss_pair, &s);
    *loss_sum = -s.sum;
    *n_pairs = h->st_pairs;
    return 0;
}
/* the same over an explicit pair list (for the finite-difference pin) */
double orc_loss_pairs(orc *h, const int32_t *centre, const int32_t *context, const int32_t *negs,
                      uint64_t P, uint32_t N)
{
    lossctx s = { h, 0.0 };
    for (uint64_t p = 0; p < P; ++p) loss_pair(&s, p, centre[p], context[p], negs + p * N, N);
    return -s.sum;
}

/* ------------------------------------------------------------------ */
/* Continuous bag of words (footnote to Section 5).                     */
/* One example per kept token q that has at least one context word:     */
/*   hbar = mean over the window's context words k of u(w_k)            */
/*   targets: the centre word w_q (label 1) and N negatives != w_q      */
/*   f = hbar . v(t),  g = lr (label - sigma(f))                        */
/*   v(t) += g hbar;   every context word: u(w_k) += (sum_t g v(t)) / |C| */
/* i.e. plus lr times the exact gradient of                             */
/*   log s(hbar.v(w_q)) + sum_neg log s(-hbar.v(neg)).                  */
/* Window and sub-sampling as in the skip-gram step; the negatives use  */
/* the counter slot of offset 0 (slot = W), which no skip-gram pair has. */
/* ------------------------------------------------------------------ */
typedef void (*cbow_fn)(void *ctx, uint64_t ex_index, int32_t centre, const int32_t *contexts,
                        uint32_t n_ctx, const int32_t *negs, uint32_t N);

static void sample_chunk_cbow(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N,
                              uint64_t step_id, cbow_fn fn, void *ctx)
{
    uint32_t k0 = (uint32_t)h->seed;
    uint32_t k1 = (uint32_t)(h->seed >> 32) ^ (uint32_t)(step_id >> 32);
    uint32_t step_lo = (uint32_t)step_id;
    if (h->cap_kept < n + 1) {
        free(h->ctok); free(h->cidx); free(h->csent);
        h->cap_kept = n + 1;
        h->ctok = (int32_t *)malloc(h->cap_kept * sizeof(int32_t));
        h->cidx = (uint32_t *)malloc(h->cap_kept * sizeof(uint32_t));
        h->csent = (uint32_t *)malloc(h->cap_kept * sizeof(uint32_t));
    }
    h->st_tokens = n; h->st_kept = h->st_centres = h->st_pairs = 0;
    h->st_draws = h->st_redraws = h->st_oov = 0;
    uint64_t nk = 0;
    uint32_t sent = 0;
    for (uint64_t i = 0; i < n; ++i) {
        int32_t w = tokens[i];
        if (w == -1) { sent++; continue; }
        if (w < 0 || (uint64_t)w >= h->vocab) { h->st_oov++; continue; }
        uint32_t thr = h->keep_thr[w];
        if (thr != 0xFFFFFFFFu) {
            uint32_t r[4];
            philox4x32_10(k0, k1, (uint32_t)i, step_lo, PUR_SUBSAMPLE, 0, r);
            if (!(r[0] < thr)) continue;
        }
        h->ctok[nk] = w; h->cidx[nk] = (uint32_t)i; h->csent[nk] = sent;
        nk++;
    }
    h->st_kept = nk;

    int32_t negs[64], contexts[256];
    uint64_t ex = 0;
    for (uint64_t q = 0; q < nk; ++q) {
        uint32_t r[4];
        if (h->il_stride > 1 && h->cidx[q] % h->il_stride != h->il_phase) continue;
        philox4x32_10(k0, k1, h->cidx[q], step_lo, PUR_RADIUS, 0, r);
        int64_t b = 1 + (int64_t)(((uint64_t)r[0] * (uint64_t)W) >> 32);
        uint32_t n_ctx = 0;
        for (int64_t p = (int64_t)q - b; p <= (int64_t)q + b; ++p) {
            if (p == (int64_t)q || p < 0 || p >= (int64_t)nk) continue;
            if (h->csent[p] != h->csent[q]) continue;
            contexts[n_ctx++] = h->ctok[p];
        }
        if (n_ctx == 0) continue;
        int32_t wq = h->ctok[q];
        for (uint32_t k = 0; k < N; ++k) {
            uint32_t cand = 0;
            int found = 0;
            for (uint32_t a = 0; a < 16 && !found; ++a) {
                philox4x32_10(k0, k1, h->cidx[q], step_lo, PUR_NEGATIVE | (W << 8), k | (a << 16), r);
                cand = alias_draw(h, r);
                h->st_draws++;
                if (cand != (uint32_t)wq) found = 1; else h->st_redraws++;
            }
            if (!found) cand = (uint32_t)(((uint64_t)wq + 1) % h->vocab);
            negs[k] = (int32_t)cand;
        }
        fn(ctx, ex++, wq, contexts, n_ctx, negs, N);
        h->st_pairs += n_ctx;
    }
    h->st_centres = ex;
}

/* ---- the examples as lists: centre[E], negs[E*N], ctx_off[E+1], ctx[sum |C|] ---- */
typedef struct {
    int32_t *centre, *negs, *ctx; uint64_t *ctx_off; uint64_t cap_ex, cap_ctx, n_ctx;
} cbowsink;
static void sink_example(void *ctx, uint64_t ex, int32_t c, const int32_t *contexts, uint32_t n_ctx,
                         const int32_t *negs, uint32_t N)
{
    cbowsink *s = (cbowsink *)ctx;
    if (ex < s->cap_ex) {
        s->centre[ex] = c;
        for (uint32_t k = 0; k < N; ++k) s->negs[ex * N + k] = negs[k];
        s->ctx_off[ex] = s->n_ctx;
    }
    for (uint32_t k = 0; k < n_ctx; ++k) {
        if (s->n_ctx < s->cap_ctx) s->ctx[s->n_ctx] = contexts[k];
        s->n_ctx++;
    }
    if (ex < s->cap_ex) s->ctx_off[ex + 1] = s->n_ctx;
}
int orc_cbow_examples(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N,
                      int32_t *centre, int32_t *negs, uint64_t *ctx_off, int32_t *ctx,
                      uint64_t cap_ex, uint64_t cap_ctx, uint64_t *n_ex, uint64_t *n_ctx)
{
    if (!h->have_tables || W < 1 || W > 127 || N < 1 || N > 64) return -1;
    cbowsink s = { centre, negs, ctx, ctx_off, cap_ex, cap_ctx, 0 };
    if (cap_ex) ctx_off[0] = 0;
    sample_chunk_cbow(h, tokens, n, W, N, h->step_id, sink_example, &s);
    *n_ex = h->st_centres; *n_ctx = s.n_ctx;
    return 0;
}

static void mean_context(orc *h, const int32_t *contexts, uint32_t n_ctx, double *hbar)
{
    uint32_t d = h->d;
    for (uint32_t j = 0; j < d; ++j) hbar[j] = 0.0;
    for (uint32_t k = 0; k < n_ctx; ++k) {
        const float *u = rs_row(&h->U, h, (uint64_t)contexts[k]);
        for (uint32_t j = 0; j < d; ++j) hbar[j] += (double)u[j];
    }
    for (uint32_t j = 0; j < d; ++j) hbar[j] /= (double)n_ctx;
}
static double dot_hv(const double *hbar, const float *v, uint32_t d)
{
    double s = 0.0;
    for (uint32_t j = 0; j < d; ++j) s += hbar[j] * (double)v[j];
    return s;
}

/* -- mode 1: one example after another, each seeing all earlier writes -- */
typedef struct { orc *h; double lr; double *hbar, *e; } cseqctx;
static void cbow_seq(void *ctx, uint64_t ex, int32_t c, const int32_t *contexts, uint32_t n_ctx,
                     const int32_t *negs, uint32_t N)
{
    (void)ex;
    cseqctx *s = (cseqctx *)ctx;
    orc *h = s->h;
    uint32_t d = h->d;
    mean_context(h, contexts, n_ctx, s->hbar);
    for (uint32_t j = 0; j < d; ++j) s->e[j] = 0.0;
    for (uint32_t k = 0; k <= N; ++k) {
        int32_t t = k == 0 ? c : negs[k - 1];
        double label = k == 0 ? 1.0 : 0.0;
        float *v = rs_row(&h->V, h, (uint64_t)t);
        double g = s->lr * (label - sigmoid(dot_hv(s->hbar, v, d)));
        for (uint32_t j = 0; j < d; ++j) s->e[j] += g * (double)v[j];
        for (uint32_t j = 0; j < d; ++j) v[j] = (float)((double)v[j] + g * s->hbar[j]);
    }
    for (uint32_t k = 0; k < n_ctx; ++k) {
        float *u = rs_row(&h->U, h, (uint64_t)contexts[k]);
        for (uint32_t j = 0; j < d; ++j) u[j] = (float)((double)u[j] + s->e[j] / (double)n_ctx);
    }
}

/* -- mode 0: every read sees start-of-step values, sums applied at the end -- */
typedef struct { snapctx sn; double *hbar, *e; } csnapctx;
static void cbow_snap(void *ctx, uint64_t ex, int32_t c, const int32_t *contexts, uint32_t n_ctx,
                      const int32_t *negs, uint32_t N)
{
    (void)ex;
    csnapctx *s = (csnapctx *)ctx;
    orc *h = s->sn.h;
    uint32_t d = h->d;
    mean_context(h, contexts, n_ctx, s->hbar);
    for (uint32_t j = 0; j < d; ++j) s->e[j] = 0.0;
    for (uint32_t k = 0; k <= N; ++k) {
        int32_t t = k == 0 ? c : negs[k - 1];
        const float *v = rs_row(&h->V, h, (uint64_t)t);
        double f = dot_hv(s->hbar, v, d);
        double g = k == 0 ? s->sn.lr * (1.0 - sigmoid(f)) : -s->sn.lr * sigmoid(f);
        for (uint32_t j = 0; j < d; ++j) s->e[j] += g * (double)v[j];
        double *dv = delta_row(&s->sn, 0, t);
        for (uint32_t j = 0; j < d; ++j) dv[j] += g * s->hbar[j];
    }
    for (uint32_t k = 0; k < n_ctx; ++k) {
        double *du = delta_row(&s->sn, 1, contexts[k]);
        for (uint32_t j = 0; j < d; ++j) du[j] += s->e[j] / (double)n_ctx;
    }
}

typedef struct { orc *h; double sum; double *hbar; } clossctx;
static void cbow_loss_ex(void *ctx, uint64_t ex, int32_t c, const int32_t *contexts, uint32_t n_ctx,
                         const int32_t *negs, uint32_t N)
{
    (void)ex;
    clossctx *s = (clossctx *)ctx;
    orc *h = s->h;
    mean_context(h, contexts, n_ctx, s->hbar);
    s->sum += log_sigmoid(dot_hv(s->hbar, rs_row(&h->V, h, (uint64_t)c), h->d));
    for (uint32_t k = 0; k < N; ++k)
        s->sum += log_sigmoid(-dot_hv(s->hbar, rs_row(&h->V, h, (uint64_t)negs[k]), h->d));
}

/* runs fn over sampled examples (tokens != NULL) or over explicit lists */
static void cbow_run(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N, uint64_t step_id,
                     const int32_t *centre, const int32_t *negs, const uint64_t *ctx_off,
                     const int32_t *ctxs, uint64_t E, cbow_fn fn, void *ctx)
{
    if (tokens) { sample_chunk_cbow(h, tokens, n, W, N, step_id, fn, ctx); return; }
    for (uint64_t e = 0; e < E; ++e)
        fn(ctx, e, centre[e], ctxs + ctx_off[e], (uint32_t)(ctx_off[e + 1] - ctx_off[e]), negs + e * N, N);
}

static int cbow_step_impl(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N,
                          const int32_t *centre, const int32_t *negs, const uint64_t *ctx_off,
                          const int32_t *ctxs, uint64_t E, double lr, uint32_t mode)
{
    double *hbar = (double *)malloc(h->d * sizeof(double)), *e = (double *)malloc(h->d * sizeof(double));
    if (mode == 1) {
        cseqctx s = { h, lr, hbar, e };
        cbow_run(h, tokens, n, W, N, h->step_id, centre, negs, ctx_off, ctxs, E, cbow_seq, &s);
    } else {
        csnapctx s;
        memset(&s, 0, sizeof(s));
        s.sn.h = h; s.sn.lr = lr; s.hbar = hbar; s.e = e;
        idmap_init(&s.sn.du_map, 4096); idmap_init(&s.sn.dv_map, 4096);
        cbow_run(h, tokens, n, W, N, h->step_id, centre, negs, ctx_off, ctxs, E, cbow_snap, &s);
        snap_apply(&s.sn, 1);
        snap_apply(&s.sn, 0);
        idmap_free(&s.sn.du_map); idmap_free(&s.sn.dv_map);
        free(s.sn.du); free(s.sn.dv);
    }
    free(hbar); free(e);
    return 0;
}
int orc_cbow_step(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N, double lr, uint32_t mode)
{
    if (!h->have_tables || W < 1 || W > 127 || N < 1 || N > 64 || mode > 1) return -1;
    cbow_step_impl(h, tokens, n, W, N, NULL, NULL, NULL, NULL, 0, lr, mode);
    h->step_id++;
    return 0;
}
int orc_cbow_step_examples(orc *h, const int32_t *centre, const int32_t *negs, const uint64_t *ctx_off,
                           const int32_t *ctxs, uint64_t E, uint32_t N, double lr, uint32_t mode)
{
    if (mode > 1 || N > 64) return -1;
    return cbow_step_impl(h, NULL, 0, 0, N, centre, negs, ctx_off, ctxs, E, lr, mode);
}
int orc_cbow_loss(orc *h, const int32_t *tokens, uint64_t n, uint32_t W, uint32_t N, uint64_t step_id,
                  double *loss_sum, uint64_t *n_examples)
{
    if (!h->have_tables || W < 1 || W > 127 || N < 1 || N > 64) return -1;
    clossctx s = { h, 0.0, (double *)malloc(h->d * sizeof(double)) };
    sample_chunk_cbow(h, tokens, n, W, N, step_id, cbow_loss_ex, &s);
    free(s.hbar);
    *loss_sum = -s.sum;
    *n_examples = h->st_centres;
    return 0;
}
double orc_cbow_loss_examples(orc *h, const int32_t *centre, const int32_t *negs, const uint64_t *ctx_off,
                              const int32_t *ctxs, uint64_t E, uint32_t N)
{
    clossctx s = { h, 0.0, (double *)malloc(h->d * sizeof(double)) };
    cbow_run(h, NULL, 0, 0, N, 0, centre, negs, ctx_off, ctxs, E, cbow_loss_ex, &s);
    free(s.hbar);
    return -s.sum;
}

/* ------------------------------------------------------------------ */
/* Retrieval by cosine similarity (Section 2; Section 7.2: K = 30 nearest */
/* with cosine above tau = 0.65).  For every query row q the candidates   */
/* are the rows cand_lo <= a < cand_hi, a != q; cos(q, a) = x_q.x_a /      */
/* (|x_q| |x_a|) in fp64 (0 if either norm is 0).  Kept: cos > tau; of    */
/* those the K largest, by decreasing cosine, ties by increasing id.       */
/* out_ids is padded with -1 and out_cos with 0.                           */
/* ------------------------------------------------------------------ */
int orc_topk_cosine(orc *h, uint32_t which, const int64_t *queries, uint64_t m, uint64_t cand_lo,
                    uint64_t cand_hi, uint32_t K, double tau, int64_t *out_ids, double *out_cos)
{
    if (which > 1 || K < 1 || cand_lo > cand_hi || cand_hi > h->vocab) return -1;
    rowstore *rs = which ? &h->V : &h->U;
    uint32_t d = h->d;
    uint64_t nc = cand_hi - cand_lo;
    double *norm = (double *)malloc((nc ? nc : 1) * sizeof(double));
    for (uint64_t a = 0; a < nc; ++a) {
        const float *x = rs_row(rs, h, cand_lo + a);
        double s = 0.0;
        for (uint32_t j = 0; j < d; ++j) s += (double)x[j] * (double)x[j];
        norm[a] = sqrt(s);
    }
    for (uint64_t i = 0; i < m; ++i) {
        int64_t *ids = out_ids + i * K;
        double *cs = out_cos + i * K;
        for (uint32_t k = 0; k < K; ++k) { ids[k] = -1; cs[k] = 0.0; }
        int64_t q = queries[i];
        if (q < 0 || (uint64_t)q >= h->vocab) continue;
        const float *xq = rs_row(rs, h, (uint64_t)q);
        double nq = 0.0;
        for (uint32_t j = 0; j < d; ++j) nq += (double)xq[j] * (double)xq[j];
        nq = sqrt(nq);
        uint32_t have = 0;
        for (uint64_t a = 0; a < nc; ++a) {
            if ((int64_t)(cand_lo + a) == q) continue;
            const float *xa = rs_row(rs, h, cand_lo + a);
            double c = 0.0;
            if (nq > 0.0 && norm[a] > 0.0) c = dot_rows(xq, xa, 0, d) / (nq * norm[a]);
            if (!(c > tau)) continue;
            /* insertion into the sorted list of the best K so far */
            uint32_t pos = have;
            while (pos > 0 && cs[pos - 1] < c) --pos;      /* equal cosine: the smaller id stays ahead */
            if (pos >= K) continue;
            uint32_t last = have < K ? have : K - 1;
            for (uint32_t k = last; k > pos; --k) { cs[k] = cs[k - 1]; ids[k] = ids[k - 1]; }
            cs[pos] = c; ids[pos] = (int64_t)(cand_lo + a);
            if (have < K) ++have;
        }
    }
    free(norm);
    return 0;
}

uint64_t orc_rows_resident(const orc *h, uint32_t which)
{
    const rowstore *rs = which ? &h->V : &h->U;
    return rs->sparse ? rs->n_rows : rs->vocab;
}

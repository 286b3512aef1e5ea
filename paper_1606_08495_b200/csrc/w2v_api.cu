// C-ABI layer of libw2v: argument checks, the handle, scratch management and the
// sequence of kernel launches that makes one step.  See include/w2v.h for the contract.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/w2v.h"
#include "w2v_internal.h"

using namespace w2v;

struct w2v_handle {
    uint64_t vocab = 0;
    uint32_t d = 0;
    uint32_t ld = 0;                 // row stride of U and V in floats (>= d, a multiple of 4)
    uint32_t d_full = 0;             // columns of the whole vectors (== d unless this is a column shard)
    uint32_t col_lo = 0;             // first column held (0 unless this is a column shard)
    bool is_shard = false;
    // state between w2v_shard_dots and w2v_shard_adjust
    bool shard_pending = false;
    int32_t *l_centre = nullptr, *l_context = nullptr, *l_negs = nullptr;   // pair list of a narrow shard's step
    uint64_t l_cap_pairs = 0, l_cap_context = 0, l_cap_negs = 0;
    float *inv_norm = nullptr; uint64_t inv_norm_cap = 0;                      // retrieval scratch
    float *part_cos = nullptr; long long *part_ids = nullptr; uint64_t part_cap = 0;
    uint32_t retrieval_kernel = 2;       // 0: fp32 on the CUDA cores, 1: tensor cores (3 x TF32), 2: tensor-core screen + exact fp32, 3: the screen on pairs of SMs
    int *tc_error = nullptr;             // device word raised by a tensor-core block whose wait ran out
    unsigned char *qsplit = nullptr; uint64_t qsplit_cap = 0;   // query rows split into TF32 head and tail
    unsigned char *ctiles = nullptr; uint64_t ctiles_cap = 0;   // candidate rows packed as bf16 operand blocks (screening kernel)
    unsigned int *floor_q = nullptr; uint64_t floor_cap = 0;    // per query: best K-th cosine reached by any block (screening kernel)
    uint32_t pend_window = 0, pend_negatives = 0;
    uint64_t pend_n = 0, pend_pairs = 0;
    uint64_t seed = 0;
    uint64_t step_id = 0;
    uint32_t il_phase = 0, il_stride = 1;   // interleaved minibatches: which tokens are input words
    int device = 0;
    int sms = 148;
    cudaStream_t stream = nullptr;
    float *U = nullptr, *V = nullptr;
    bool owns_tables = false;
    // sampling tables
    uint32_t *keep_thr = nullptr;
    uint2 *alias = nullptr;
    bool have_tables = false;
    // scratch
    Scratch sc;
    DevState *st = nullptr;          // device
    DevState *st_host = nullptr;     // pinned mirror
    float *G = nullptr;
    uint64_t G_cap = 0;
    float *DU = nullptr;
    uint64_t DU_cap = 0;             // floats
    double *DV = nullptr;            // fp64 sums for the most-hit output rows (snapshot mode), kept zero between steps
    uint64_t DV_cap = 0;             // doubles
    uint32_t hot_rows = 0;
    int32_t *tok_stage = nullptr;
    uint64_t tok_stage_cap = 0;
    // tuning / accounting
    uint32_t rows_in_flight = 0, blocks_per_sm = 0;
    uint64_t launches = 0;
    bool profiling = false;
    std::vector<cudaEvent_t> ev;     // pairs (start, stop)
    size_t ev_used = 0;
    double prof_ms = 0.0;
    uint64_t prof_launches = 0;
    char err[256] = "no error";
};

namespace {

int32_t fail(w2v_handle *h, int32_t code, const char *what, cudaError_t ce = cudaSuccess)
{
    if (h) {
        if (ce != cudaSuccess)
            std::snprintf(h->err, sizeof(h->err), "%s: %s", what, cudaGetErrorString(ce));
        else
            std::snprintf(h->err, sizeof(h->err), "%s", what);
    }
    return code;
}

#define W2V_CUDA(h, call)                                                     \
    do {                                                                      \
        cudaError_t ce_ = (call);                                             \
        if (ce_ != cudaSuccess)                                               \
            return fail(h, ce_ == cudaErrorMemoryAllocation ? W2V_ERR_NOMEM : W2V_ERR_CUDA, #call, ce_); \
    } while (0)

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) { cudaGetDevice(&prev); if (prev != dev) cudaSetDevice(dev); else prev = -1; }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

template <typename T>
cudaError_t dev_alloc(T **p, uint64_t count)
{
    return cudaMalloc(reinterpret_cast<void **>(p), (count ? count : 1) * sizeof(T));
}

void free_scratch(Scratch &sc)
{
    cudaFree(sc.flags); cudaFree(sc.tile_sums); cudaFree(sc.tile_offs); cudaFree(sc.ctok);
    cudaFree(sc.cidx); cudaFree(sc.csent); cudaFree(sc.win); cudaFree(sc.cnt_tile); cudaFree(sc.pair_off);
    sc = Scratch();
}

// Scratch for chunks of up to n tokens; grows only.
int32_t ensure_scratch(w2v_handle *h, uint64_t n)
{
    if (n <= h->sc.n_cap) return W2V_OK;
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    free_scratch(h->sc);
    const uint64_t tiles = (n + kScanTile - 1) / kScanTile + 1;
    Scratch &sc = h->sc;
    W2V_CUDA(h, dev_alloc(&sc.flags, n));
    W2V_CUDA(h, dev_alloc(&sc.tile_sums, tiles));
    W2V_CUDA(h, dev_alloc(&sc.tile_offs, tiles));
    W2V_CUDA(h, dev_alloc(&sc.ctok, n));
    W2V_CUDA(h, dev_alloc(&sc.cidx, n));
    W2V_CUDA(h, dev_alloc(&sc.csent, n));
    W2V_CUDA(h, dev_alloc(&sc.win, n));
    W2V_CUDA(h, dev_alloc(&sc.cnt_tile, tiles));
    W2V_CUDA(h, dev_alloc(&sc.pair_off, n + 1));
    sc.n_cap = n;
    return W2V_OK;
}

// Makes *p hold at least `need` elements.  When it does not, the stream is drained (it may still
// use the old array), the array is freed and a new one allocated; with `slack`, a quarter more than
// asked for, so that chunks of slightly different sizes do not re-allocate every time.
template <typename T>
int32_t grow(w2v_handle *h, T **p, uint64_t *cap, uint64_t need, bool slack)
{
    if (need <= *cap) return W2V_OK;
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    cudaFree(*p); *p = nullptr; *cap = 0;
    const uint64_t want = slack ? need + need / 4 + 1024 : need;
    W2V_CUDA(h, dev_alloc(p, want));
    *cap = want;
    return W2V_OK;
}

// Scratch of the deferred-update passes (Algorithm 2 applies its updates only when the call ends):
// coefficients G for `targets` targets, per-centre sums DU for every token the chunk scratch holds,
// fp64 sums DV of the most-hit output rows (zero between steps).
int32_t ensure_update_scratch(w2v_handle *h, uint64_t targets, bool slack)
{
    int32_t rc;
    if ((rc = grow(h, &h->G, &h->G_cap, targets, slack)) != W2V_OK) return rc;
    if ((rc = grow(h, &h->DU, &h->DU_cap, h->sc.n_cap * (uint64_t)h->d, false)) != W2V_OK) return rc;
    const uint64_t need_dv = (uint64_t)h->hot_rows * h->d;
    if (need_dv > h->DV_cap) {
        if ((rc = grow(h, &h->DV, &h->DV_cap, need_dv, false)) != W2V_OK) return rc;
        W2V_CUDA(h, cudaMemsetAsync(h->DV, 0, h->DV_cap * sizeof(double), h->stream));
    }
    return W2V_OK;
}

// Copies a chunk that lives in host memory into the handle's staging array (stream-ordered).
int32_t stage_tokens(w2v_handle *h, const int32_t *tokens_host, uint64_t n)
{
    int32_t rc = grow(h, &h->tok_stage, &h->tok_stage_cap, n, false);
    if (rc != W2V_OK) return rc;
    if (n)
        W2V_CUDA(h, cudaMemcpyAsync(h->tok_stage, tokens_host, n * sizeof(int32_t), cudaMemcpyHostToDevice, h->stream));
    return W2V_OK;
}

// The device word that kernels with bounded waits raise when a wait runs out (read by w2v_sync).
int32_t ensure_error_word(w2v_handle *h)
{
    if (h->tc_error) return W2V_OK;
    W2V_CUDA(h, dev_alloc(&h->tc_error, 1));
    W2V_CUDA(h, cudaMemsetAsync(h->tc_error, 0, sizeof(int), h->stream));
    return W2V_OK;
}

// Snapshot mode sizes its per-target arrays from the bound "every token is an input word with a
// full window" when they then stay within this many bytes: the steady-state step neither waits for
// the pair count nor re-allocates.  Larger bounds (wide windows on long chunks) fall back to
// reading the pair count.
constexpr uint64_t kSnapshotBoundBudget = 1ull << 30;
constexpr uint64_t kListChunk = 500000;       // Hogwild mode: chunks of at least this many tokens use a list of negatives

int32_t check_step_args(w2v_handle *h, const void *tokens, uint64_t n, uint32_t window, uint32_t negatives)
{
    if (!h) return W2V_ERR_ARG;
    if (!tokens && n) return fail(h, W2V_ERR_ARG, "tokens is NULL");
    if (n >= (1ull << 31)) return fail(h, W2V_ERR_ARG, "n must be below 2^31");
    if (window < 1 || window > 127) return fail(h, W2V_ERR_ARG, "window must be in 1..127");
    if (negatives < 1 || negatives > 64) return fail(h, W2V_ERR_ARG, "negatives must be in 1..64");
    if (!h->have_tables) return fail(h, W2V_ERR_STATE, "w2v_build_alias has not been called");
    return W2V_OK;
}

StepParams make_params(w2v_handle *h, uint32_t window, uint32_t negatives, float lr)
{
    StepParams p;
    std::memset(&p, 0, sizeof(p));
    p.U = h->U; p.V = h->V;
    p.tab.keep_thr = h->keep_thr; p.tab.alias = h->alias;
    p.ctok = h->sc.ctok; p.cidx = h->sc.cidx; p.win = h->sc.win;
    p.st = h->st;
    p.vocab = (uint32_t)h->vocab; p.d4 = h->d / 4; p.ld4 = h->ld / 4;
    p.window = window; p.negatives = negatives;
    p.k0 = (uint32_t)h->seed;
    p.k1 = (uint32_t)(h->seed >> 32) ^ (uint32_t)(h->step_id >> 32);
    p.step_lo = (uint32_t)h->step_id;
    p.lr = lr;
    p.pair_off = h->sc.pair_off; p.G = h->G; p.DU = h->DU;
    p.DV = h->DV; p.hot_rows = h->DV ? h->hot_rows : 0;
    p.l_centre = h->l_centre; p.l_context = h->l_context; p.l_negs = h->l_negs;
    return p;
}

// sub-sampling, compaction and windows for the chunk; counters zeroed first
int32_t enqueue_sampling(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window)
{
    int32_t rc = ensure_scratch(h, n);
    if (rc != W2V_OK) return rc;
    h->shard_pending = false;            // the scratch a pending w2v_shard_adjust would need is overwritten
    const uint32_t k0 = (uint32_t)h->seed;
    const uint32_t k1 = (uint32_t)(h->seed >> 32) ^ (uint32_t)(h->step_id >> 32);
    const uint32_t step_lo = (uint32_t)h->step_id;
    SampleTables tab{h->keep_thr, h->alias};
    if (n > 0 && n <= kSmallChunk) {
        int k = launch_sample_small(tokens, n, tab, (uint32_t)h->vocab, k0, k1, step_lo, window, h->il_phase,
                                    h->il_stride, h->sc, h->st, h->stream);
        if (k < 0) return fail(h, W2V_ERR_CUDA, "sampling launch", cudaGetLastError());
        h->launches += (uint64_t)k;
        return W2V_OK;
    }
    W2V_CUDA(h, cudaMemsetAsync(h->st, 0, sizeof(DevState), h->stream));
    int k = launch_compact(tokens, n, tab, (uint32_t)h->vocab, k0, k1, step_lo, h->sc, h->st, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "compaction launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    k = launch_windows(n, window, k0, k1, step_lo, h->il_phase, h->il_stride, h->sc, h->st, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "window launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    return W2V_OK;
}

int32_t read_state(w2v_handle *h, uint64_t n, w2v_step_stats *stats)
{
    W2V_CUDA(h, cudaMemcpyAsync(h->st_host, h->st, sizeof(DevState), cudaMemcpyDeviceToHost, h->stream));
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    if (stats) {
        const DevState &s = *h->st_host;
        stats->tokens = n; stats->kept = s.n_kept; stats->centres = s.centres; stats->pairs = s.pairs;
        stats->neg_draws = s.neg_draws; stats->neg_redraws = s.neg_redraws; stats->oov = s.oov;
        stats->status = s.status; stats->reserved = 0;
    }
    return W2V_OK;
}

void profile_collect(w2v_handle *h)
{
    for (size_t i = 0; i + 1 < h->ev_used; i += 2) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, h->ev[i], h->ev[i + 1]) == cudaSuccess) h->prof_ms += ms;
    }
    h->ev_used = 0;
}

// records an event on the stream; every second call closes a (start, stop) pair
int32_t profile_mark(w2v_handle *h)
{
    if (!h->profiling) return W2V_OK;
    if (h->ev_used == h->ev.size()) {
        if (h->ev.size() >= 512) {           // recycle: wait, fold into the sum, start over
            W2V_CUDA(h, cudaStreamSynchronize(h->stream));
            profile_collect(h);
        } else {
            cudaEvent_t e;
            W2V_CUDA(h, cudaEventCreate(&e));
            h->ev.push_back(e);
        }
    }
    W2V_CUDA(h, cudaEventRecord(h->ev[h->ev_used++], h->stream));
    return W2V_OK;
}

int32_t step_impl(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window, uint32_t negatives,
                  float lr, uint32_t mode, w2v_step_stats *stats)
{
    if (mode > 1) return fail(h, W2V_ERR_ARG, "mode must be 0 (snapshot) or 1 (hogwild)");
    if (h->is_shard)
        return fail(h, W2V_ERR_STATE, "a column shard steps through w2v_shard_dots and w2v_shard_adjust");
    int32_t rc = enqueue_sampling(h, tokens, n, window);
    if (rc != W2V_OK) return rc;
    if (mode == W2V_MODE_HOGWILD) {
        // long chunks draw their negatives into a list first (four more launches, a faster update
        // kernel: measured equal on the device at 0.26 M tokens but slower end to end, 6 % faster at 1 M tokens with 5 negatives), when
        // the list for the worst case fits the budget
        const uint64_t negs_cap = n * 2ull * window * negatives;
        const bool list = n >= kListChunk && negs_cap * sizeof(int32_t) <= kSnapshotBoundBudget;
        if (list) {
            int k = launch_pair_offsets(n, h->sc, h->st, h->stream);
            if (k < 0) return fail(h, W2V_ERR_CUDA, "pair offset launch", cudaGetLastError());
            h->launches += (uint64_t)k;
            if ((rc = grow(h, &h->l_negs, &h->l_cap_negs, negs_cap, false)) != W2V_OK) return rc;
        }
        StepParams p = make_params(h, window, negatives, lr);
        p.keep_negs = list ? 1u : 0u;
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
        int k = launch_hogwild(p, h->rows_in_flight, h->blocks_per_sm, h->sms, h->stream);
        if (k < 0) return fail(h, W2V_ERR_CUDA, "update kernel launch", cudaGetLastError());
        h->launches += (uint64_t)k;
        if (h->profiling) h->prof_launches += (uint64_t)k;
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
    } else {
        int k = launch_pair_offsets(n, h->sc, h->st, h->stream);
        if (k < 0) return fail(h, W2V_ERR_CUDA, "pair offset launch", cudaGetLastError());
        h->launches += (uint64_t)k;
        // G and the list of negatives (drawn in pass 1, read back instead of drawn again in pass 2) hold
        // one entry per target / per negative: sized from the bound when that is affordable, else
        // from the pair count, which only the device knows
        uint64_t pairs_cap = n * 2ull * window;
        const bool bounded = pairs_cap * (2ull * negatives + 1ull) * sizeof(float) <= kSnapshotBoundBudget;
        if (!bounded) {
            if ((rc = read_state(h, n, nullptr)) != W2V_OK) return rc;
            pairs_cap = h->st_host->pairs;
        }
        if ((rc = ensure_update_scratch(h, pairs_cap * (uint64_t)(negatives + 1), !bounded)) != W2V_OK) return rc;
        if ((rc = grow(h, &h->l_negs, &h->l_cap_negs, pairs_cap * (uint64_t)negatives, !bounded)) != W2V_OK) return rc;
        if (pairs_cap > 0) {
            StepParams p = make_params(h, window, negatives, lr);
            p.keep_negs = 1u;
            if ((rc = profile_mark(h)) != W2V_OK) return rc;
            k = launch_snapshot(p, h->rows_in_flight, h->blocks_per_sm, h->sms, h->stream);
            if (k < 0) return fail(h, W2V_ERR_CUDA, "update kernel launch", cudaGetLastError());
            h->launches += (uint64_t)k;
            if (h->profiling) h->prof_launches += (uint64_t)k;
            if ((rc = profile_mark(h)) != W2V_OK) return rc;
        }
    }
    h->step_id += 1;
    if (stats) {
        if ((rc = read_state(h, n, stats)) != W2V_OK) return rc;
        if (stats->status & 2u) return fail(h, W2V_ERR_CUDA, "a copy into shared memory did not arrive in time; the step is incomplete");
        if (stats->status & 1u) return fail(h, W2V_ERR_TOKEN_RANGE, "token ids outside [-1, vocab) were skipped");
    }
    return W2V_OK;
}

// the continuous-bag-of-words step: same sampling, one example per centre with a context
int32_t cbow_step_impl(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window, uint32_t negatives,
                       float lr, uint32_t mode, w2v_step_stats *stats)
{
    if (mode > 1) return fail(h, W2V_ERR_ARG, "mode must be 0 (snapshot) or 1 (hogwild)");
    if (h->is_shard) return fail(h, W2V_ERR_STATE, "a column shard has no continuous-bag-of-words step");
    int32_t rc = enqueue_sampling(h, tokens, n, window);
    if (rc != W2V_OK) return rc;
    if (mode == W2V_MODE_HOGWILD) {
        StepParams p = make_params(h, window, negatives, lr);
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
        int k = launch_cbow_hogwild(p, h->blocks_per_sm, h->sms, h->stream);
        if (k < 0) return fail(h, W2V_ERR_CUDA, "update kernel launch", cudaGetLastError());
        h->launches += (uint64_t)k;
        if (h->profiling) h->prof_launches += (uint64_t)k;
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
    } else {
        // coefficients and kept negatives are indexed by kept position: at most one example per token
        if ((rc = ensure_update_scratch(h, n * (uint64_t)(negatives + 1), false)) != W2V_OK) return rc;
        if ((rc = grow(h, &h->l_negs, &h->l_cap_negs, n * (uint64_t)negatives, false)) != W2V_OK) return rc;
        if (n > 0) {
            StepParams p = make_params(h, window, negatives, lr);
            p.keep_negs = 1u;
            if ((rc = profile_mark(h)) != W2V_OK) return rc;
            int k = launch_cbow_snapshot(p, h->blocks_per_sm, h->sms, h->stream);
            if (k < 0) return fail(h, W2V_ERR_CUDA, "update kernel launch", cudaGetLastError());
            h->launches += (uint64_t)k;
            if (h->profiling) h->prof_launches += (uint64_t)k;
            if ((rc = profile_mark(h)) != W2V_OK) return rc;
        }
    }
    h->step_id += 1;
    if (stats) {
        if ((rc = read_state(h, n, stats)) != W2V_OK) return rc;
        if (stats->status & 1u) return fail(h, W2V_ERR_TOKEN_RANGE, "token ids outside [-1, vocab) were skipped");
    }
    return W2V_OK;
}

}  // namespace

extern "C" {

int32_t w2v_create(uint64_t vocab, uint32_t d, uint64_t seed, float *U, float *V, void *stream,
                   w2v_handle **out)
{
    return w2v_create_strided(vocab, d, d, seed, U, V, stream, out);
}

int32_t w2v_create_strided(uint64_t vocab, uint32_t d, uint32_t row_stride, uint64_t seed, float *U, float *V,
                           void *stream, w2v_handle **out)
{
    return w2v_create_shard(vocab, d, 0, d, row_stride, seed, U, V, stream, out);
}

int32_t w2v_create_shard(uint64_t vocab, uint32_t d_full, uint32_t col_lo, uint32_t col_hi, uint32_t row_stride,
                         uint64_t seed, float *U, float *V, void *stream, w2v_handle **out)
{
    if (!out) return W2V_ERR_ARG;
    *out = nullptr;
    if (vocab < 2 || vocab >= (1ull << 31)) return W2V_ERR_ARG;
    if (d_full < 4 || d_full > 1024 || (d_full % 4) != 0) return W2V_ERR_ARG;
    if (!(col_lo < col_hi && col_hi <= d_full) || (col_lo % 4) != 0 || (col_hi % 4) != 0) return W2V_ERR_ARG;
    const uint32_t d = col_hi - col_lo;
    if (row_stride < d || row_stride > 2048 || (row_stride % 4) != 0) return W2V_ERR_ARG;
    if ((U == nullptr) != (V == nullptr)) return W2V_ERR_ARG;
    if (U && ((reinterpret_cast<uintptr_t>(U) | reinterpret_cast<uintptr_t>(V)) & 15u)) return W2V_ERR_ARG;
    w2v_handle *h = new (std::nothrow) w2v_handle();
    if (!h) return W2V_ERR_NOMEM;
    h->vocab = vocab; h->d = d; h->ld = row_stride; h->seed = seed;
    h->d_full = d_full; h->col_lo = col_lo; h->is_shard = d != d_full;
    h->stream = static_cast<cudaStream_t>(stream);
    auto bail = [&](int32_t code) { w2v_destroy(h); return code; };
    if (cudaGetDevice(&h->device) != cudaSuccess) return bail(W2V_ERR_CUDA);
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device) == cudaSuccess && sms > 0)
        h->sms = sms;
    const uint64_t elems = vocab * (uint64_t)row_stride;
    if (!U) {
        if (dev_alloc(&h->U, elems) != cudaSuccess) { cudaGetLastError(); return bail(W2V_ERR_NOMEM); }
        h->owns_tables = true;
        if (dev_alloc(&h->V, elems) != cudaSuccess) { cudaGetLastError(); return bail(W2V_ERR_NOMEM); }
    } else {
        h->U = U; h->V = V;
    }
    if (dev_alloc(&h->st, 1) != cudaSuccess) return bail(W2V_ERR_NOMEM);
    if (cudaMallocHost(reinterpret_cast<void **>(&h->st_host), sizeof(DevState)) != cudaSuccess)
        return bail(W2V_ERR_NOMEM);
    if (cudaMemsetAsync(h->st, 0, sizeof(DevState), h->stream) != cudaSuccess) return bail(W2V_ERR_CUDA);
    if (launch_init_tables(h->U, h->V, vocab, d, row_stride, d_full, col_lo, seed, h->stream) < 0) return bail(W2V_ERR_CUDA);
    h->launches += 1;
    *out = h;
    return W2V_OK;
}

int32_t w2v_destroy(w2v_handle *h)
{
    if (!h) return W2V_OK;
    DeviceGuard g(h->device);
    cudaStreamSynchronize(h->stream);
    if (h->owns_tables) { cudaFree(h->U); cudaFree(h->V); }
    cudaFree(h->keep_thr); cudaFree(h->alias);
    free_scratch(h->sc);
    cudaFree(h->st);
    if (h->st_host) cudaFreeHost(h->st_host);
    cudaFree(h->G); cudaFree(h->DU); cudaFree(h->DV); cudaFree(h->tok_stage);
    cudaFree(h->l_centre); cudaFree(h->l_context); cudaFree(h->l_negs);
    cudaFree(h->inv_norm); cudaFree(h->part_cos); cudaFree(h->part_ids); cudaFree(h->tc_error); cudaFree(h->qsplit); cudaFree(h->ctiles); cudaFree(h->floor_q);
    for (cudaEvent_t e : h->ev) cudaEventDestroy(e);
    cudaGetLastError();
    delete h;
    return W2V_OK;
}

int32_t w2v_build_alias(w2v_handle *h, const uint64_t *counts, double subsample_t)
{
    if (!h) return W2V_ERR_ARG;
    if (!counts) return fail(h, W2V_ERR_ARG, "counts is NULL");
    DeviceGuard g(h->device);
    std::vector<uint2> ta;
    std::vector<uint32_t> keep;
    try {
        ta.resize(h->vocab);
        keep.resize(h->vocab);
    } catch (const std::bad_alloc &) {
        return fail(h, W2V_ERR_NOMEM, "host memory for the sampling tables");
    }
    int rc;
    try {
        rc = build_tables_host(counts, h->vocab, subsample_t, ta.data(), keep.data(), &h->hot_rows);
    } catch (const std::bad_alloc &) {
        return fail(h, W2V_ERR_NOMEM, "host memory for the sampling tables");
    }
    if (rc != 0) return fail(h, W2V_ERR_ARG, "every count must be at least 1");
    if (!h->alias) W2V_CUDA(h, dev_alloc(&h->alias, h->vocab));
    if (!h->keep_thr) W2V_CUDA(h, dev_alloc(&h->keep_thr, h->vocab));
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    W2V_CUDA(h, cudaMemcpyAsync(h->alias, ta.data(), h->vocab * sizeof(uint2), cudaMemcpyHostToDevice, h->stream));
    W2V_CUDA(h, cudaMemcpyAsync(h->keep_thr, keep.data(), h->vocab * sizeof(uint32_t), cudaMemcpyHostToDevice, h->stream));
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    h->have_tables = true;
    return W2V_OK;
}

int32_t w2v_get_tables(w2v_handle *h, uint32_t *thr, uint32_t *alias, uint32_t *keep_thr)
{
    if (!h) return W2V_ERR_ARG;
    if (!h->have_tables) return fail(h, W2V_ERR_STATE, "w2v_build_alias has not been called");
    DeviceGuard g(h->device);
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    if (thr || alias) {
        std::vector<uint2> ta(h->vocab);
        W2V_CUDA(h, cudaMemcpy(ta.data(), h->alias, h->vocab * sizeof(uint2), cudaMemcpyDeviceToHost));
        for (uint64_t w = 0; w < h->vocab; ++w) {
            if (thr) thr[w] = ta[w].x;
            if (alias) alias[w] = ta[w].y;
        }
    }
    if (keep_thr)
        W2V_CUDA(h, cudaMemcpy(keep_thr, h->keep_thr, h->vocab * sizeof(uint32_t), cudaMemcpyDeviceToHost));
    return W2V_OK;
}

int32_t w2v_sgns_step(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window, uint32_t negatives,
                      float lr, uint32_t mode, w2v_step_stats *stats)
{
    int32_t rc = check_step_args(h, tokens, n, window, negatives);
    if (rc != W2V_OK) return rc;
    DeviceGuard g(h->device);
    return step_impl(h, tokens, n, window, negatives, lr, mode, stats);
}

int32_t w2v_sgns_step_host(w2v_handle *h, const int32_t *tokens_host, uint64_t n, uint32_t window,
                           uint32_t negatives, float lr, uint32_t mode, w2v_step_stats *stats)
{
    int32_t rc = check_step_args(h, tokens_host, n, window, negatives);
    if (rc != W2V_OK) return rc;
    DeviceGuard g(h->device);
    if ((rc = stage_tokens(h, tokens_host, n)) != W2V_OK) return rc;
    return step_impl(h, h->tok_stage, n, window, negatives, lr, mode, stats);
}

int32_t w2v_sample_pairs(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window, uint32_t negatives,
                         int32_t *centre, int32_t *context, int32_t *negs, uint64_t cap, uint64_t *n_pairs,
                         w2v_step_stats *stats)
{
    int32_t rc = check_step_args(h, tokens, n, window, negatives);
    if (rc != W2V_OK) return rc;
    if (!n_pairs) return fail(h, W2V_ERR_ARG, "n_pairs is NULL");
    if (cap && (!centre || !context || !negs)) return fail(h, W2V_ERR_ARG, "output array is NULL");
    DeviceGuard g(h->device);
    if ((rc = enqueue_sampling(h, tokens, n, window)) != W2V_OK) return rc;
    int k = launch_pair_offsets(n, h->sc, h->st, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "pair offset launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    if (n) {
        StepParams p = make_params(h, window, negatives, 0.f);
        k = launch_emit_pairs(p, centre, context, negs, cap, h->sms * 8, h->stream);
        if (k < 0) return fail(h, W2V_ERR_CUDA, "pair list launch", cudaGetLastError());
        h->launches += (uint64_t)k;
    }
    w2v_step_stats local;
    if ((rc = read_state(h, n, &local)) != W2V_OK) return rc;
    if (stats) *stats = local;
    *n_pairs = local.pairs;
    if (local.pairs > cap) return fail(h, W2V_ERR_CAPACITY, "more pairs than the output arrays hold");
    if (local.status & 1u) return fail(h, W2V_ERR_TOKEN_RANGE, "token ids outside [-1, vocab) were skipped");
    return W2V_OK;
}

int32_t w2v_cbow_step(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window, uint32_t negatives,
                      float lr, uint32_t mode, w2v_step_stats *stats)
{
    int32_t rc = check_step_args(h, tokens, n, window, negatives);
    if (rc != W2V_OK) return rc;
    DeviceGuard g(h->device);
    return cbow_step_impl(h, tokens, n, window, negatives, lr, mode, stats);
}

int32_t w2v_cbow_step_host(w2v_handle *h, const int32_t *tokens_host, uint64_t n, uint32_t window,
                           uint32_t negatives, float lr, uint32_t mode, w2v_step_stats *stats)
{
    int32_t rc = check_step_args(h, tokens_host, n, window, negatives);
    if (rc != W2V_OK) return rc;
    DeviceGuard g(h->device);
    if ((rc = stage_tokens(h, tokens_host, n)) != W2V_OK) return rc;
    return cbow_step_impl(h, h->tok_stage, n, window, negatives, lr, mode, stats);
}

int32_t w2v_sample_cbow(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window, uint32_t negatives,
                        int32_t *centre, int32_t *negs, uint64_t cap, uint64_t *n_examples, w2v_step_stats *stats)
{
    int32_t rc = check_step_args(h, tokens, n, window, negatives);
    if (rc != W2V_OK) return rc;
    if (!n_examples) return fail(h, W2V_ERR_ARG, "n_examples is NULL");
    if (cap && (!centre || !negs)) return fail(h, W2V_ERR_ARG, "output array is NULL");
    DeviceGuard g(h->device);
    if ((rc = enqueue_sampling(h, tokens, n, window)) != W2V_OK) return rc;
    int k = launch_pair_offsets(n, h->sc, h->st, h->stream, true);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "example offset launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    if (n) {
        StepParams p = make_params(h, window, negatives, 0.f);
        k = launch_cbow_emit(p, centre, negs, cap, h->sms * 8, h->stream);
        if (k < 0) return fail(h, W2V_ERR_CUDA, "example list launch", cudaGetLastError());
        h->launches += (uint64_t)k;
    }
    w2v_step_stats local;
    if ((rc = read_state(h, n, &local)) != W2V_OK) return rc;
    if (stats) *stats = local;
    *n_examples = local.centres;
    if (local.centres > cap) return fail(h, W2V_ERR_CAPACITY, "more examples than the output arrays hold");
    if (local.status & 1u) return fail(h, W2V_ERR_TOKEN_RANGE, "token ids outside [-1, vocab) were skipped");
    return W2V_OK;
}

int32_t w2v_shard_dots(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window, uint32_t negatives,
                       float *const *F_peers, uint32_t n_peers, uint64_t cap, w2v_step_stats *stats)
{
    int32_t rc = check_step_args(h, tokens, n, window, negatives);
    if (rc != W2V_OK) return rc;
    if (!F_peers || n_peers < 1 || n_peers > (uint32_t)kMaxShards)
        return fail(h, W2V_ERR_ARG, "need between 1 and 16 arrays for the partial dot products");
    ShardPeers peers;
    std::memset(&peers, 0, sizeof(peers));
    for (uint32_t r = 0; r < n_peers; ++r) {
        if (!F_peers[r]) return fail(h, W2V_ERR_ARG, "an array for the partial dot products is NULL");
        peers.F[r] = F_peers[r];
    }
    peers.n = n_peers;
    DeviceGuard g(h->device);
    if ((rc = enqueue_sampling(h, tokens, n, window)) != W2V_OK) return rc;
    int k = launch_pair_offsets(n, h->sc, h->st, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "pair offset launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    if ((rc = read_state(h, n, nullptr)) != W2V_OK) return rc;      // the pair count sizes everything below
    const uint64_t pairs = h->st_host->pairs;
    if (pairs * (uint64_t)(negatives + 1) > cap)
        return fail(h, W2V_ERR_CAPACITY, "more targets than the arrays for the partial dot products hold");
    if (pairs > 0 && h->d / 4 <= kNarrowD4) {
        // narrow slice: write the index sets once, the three passes stream over them
        if ((rc = grow(h, &h->l_centre, &h->l_cap_pairs, pairs, true)) != W2V_OK) return rc;
        if ((rc = grow(h, &h->l_context, &h->l_cap_context, pairs, true)) != W2V_OK) return rc;
        if ((rc = grow(h, &h->l_negs, &h->l_cap_negs, pairs * (uint64_t)negatives, true)) != W2V_OK) return rc;
        StepParams pl = make_params(h, window, negatives, 0.f);
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
        k = launch_pair_list(pl, h->l_centre, h->l_context, h->l_negs, h->sms * 8, h->stream);
        if (k < 0) return fail(h, W2V_ERR_CUDA, "pair list launch", cudaGetLastError());
        h->launches += (uint64_t)k;
        if (h->profiling) h->prof_launches += (uint64_t)k;
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
    }
    if (pairs > 0) {
        StepParams p = make_params(h, window, negatives, 0.f);
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
        k = launch_shard_dots(p, peers, h->sms, h->stream);
        if (k < 0) return fail(h, W2V_ERR_CUDA, "partial dots launch", cudaGetLastError());
        h->launches += (uint64_t)k;
        if (h->profiling) h->prof_launches += (uint64_t)k;
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
    }
    h->shard_pending = true;
    h->pend_window = window; h->pend_negatives = negatives; h->pend_n = n; h->pend_pairs = pairs;
    if (stats) {
        if ((rc = read_state(h, n, stats)) != W2V_OK) return rc;
        if (stats->status & 1u) return fail(h, W2V_ERR_TOKEN_RANGE, "token ids outside [-1, vocab) were skipped");
    }
    return W2V_OK;
}

int32_t w2v_shard_adjust(w2v_handle *h, const float *F, float lr)
{
    if (!h) return W2V_ERR_ARG;
    if (!h->shard_pending) return fail(h, W2V_ERR_STATE, "w2v_shard_adjust needs the w2v_shard_dots call of the same step before it");
    const uint64_t targets = h->pend_pairs * (uint64_t)(h->pend_negatives + 1);
    if (targets && !F) return fail(h, W2V_ERR_ARG, "F is NULL");
    DeviceGuard g(h->device);
    int32_t rc;
    if ((rc = ensure_update_scratch(h, targets, true)) != W2V_OK) return rc;
    if (targets) {
        StepParams p = make_params(h, h->pend_window, h->pend_negatives, lr);
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
        int k = launch_shard_coefficients(F, h->G, targets, h->pend_negatives + 1, lr, h->sms, h->stream);
        int k2 = k < 0 ? -1 : launch_shard_du(p, h->sms, h->stream);
        int k3 = k2 < 0 ? -1 : launch_shard_apply(p, h->blocks_per_sm, h->sms, h->stream);
        if (k3 < 0) return fail(h, W2V_ERR_CUDA, "adjust launch", cudaGetLastError());
        h->launches += (uint64_t)(k + k2 + k3);
        if (h->profiling) h->prof_launches += (uint64_t)(k + k2 + k3);
        if ((rc = profile_mark(h)) != W2V_OK) return rc;
    }
    h->shard_pending = false;
    h->step_id += 1;
    return W2V_OK;
}

int32_t w2v_peer_barrier(w2v_handle *h, uint32_t *const *flags_peers, uint32_t n_peers, uint32_t rank,
                         uint32_t epoch, uint32_t timeout_ms)
{
    if (!h) return W2V_ERR_ARG;
    if (!flags_peers || n_peers < 1 || n_peers > (uint32_t)kMaxShards || rank >= n_peers)
        return fail(h, W2V_ERR_ARG, "need between 1 and 16 epoch arrays and rank < n_peers");
    if (timeout_ms < 1 || timeout_ms > 600000u) return fail(h, W2V_ERR_ARG, "timeout_ms must be in 1..600000");
    PeerFlags flags;
    std::memset(&flags, 0, sizeof(flags));
    for (uint32_t r = 0; r < n_peers; ++r) {
        if (!flags_peers[r] || (reinterpret_cast<uintptr_t>(flags_peers[r]) & 3u))
            return fail(h, W2V_ERR_ARG, "an epoch array is NULL or not 4-byte aligned");
        flags.p[r] = flags_peers[r];
    }
    flags.n = n_peers;
    DeviceGuard g(h->device);
    int32_t rc;
    if ((rc = ensure_error_word(h)) != W2V_OK) return rc;
    const int k = launch_peer_barrier(flags, rank, epoch, timeout_ms, h->tc_error, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "barrier launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    return W2V_OK;
}

int32_t w2v_partial_dots(w2v_handle *h, const int32_t *pairs, uint64_t m, uint32_t col_lo, uint32_t col_hi,
                         float *out)
{
    if (!h) return W2V_ERR_ARG;
    if (m && (!pairs || !out)) return fail(h, W2V_ERR_ARG, "pairs or out is NULL");
    if (!(col_lo < col_hi && col_hi <= h->d)) return fail(h, W2V_ERR_ARG, "need 0 <= col_lo < col_hi <= d");
    DeviceGuard g(h->device);
    int k = launch_partial_dots(h->U, h->V, (uint32_t)h->vocab, h->ld, pairs, m, col_lo, col_hi, out, h->st,
                                h->sms, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "partial dots launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    return W2V_OK;
}

static int32_t copy_rows(w2v_handle *h, uint32_t which, const int64_t *ids, uint64_t m, float *buf, bool to_table)
{
    if (!h) return W2V_ERR_ARG;
    if (which > 1) return fail(h, W2V_ERR_ARG, "which must be 0 (U) or 1 (V)");
    if (m && (!ids || !buf)) return fail(h, W2V_ERR_ARG, "ids or buffer is NULL");
    if (reinterpret_cast<uintptr_t>(buf) & 15u) return fail(h, W2V_ERR_ARG, "row buffer must be 16-byte aligned");
    DeviceGuard g(h->device);
    int k = launch_copy_rows(which ? h->V : h->U, (uint32_t)h->vocab, h->d, h->ld, ids, m, buf, to_table, h->sms,
                             h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "row copy launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    return W2V_OK;
}

int32_t w2v_read_rows(w2v_handle *h, uint32_t which, const int64_t *ids, uint64_t m, float *out)
{
    return copy_rows(h, which, ids, m, out, false);
}

int32_t w2v_write_rows(w2v_handle *h, uint32_t which, const int64_t *ids, uint64_t m, const float *in)
{
    return copy_rows(h, which, ids, m, const_cast<float *>(in), true);
}

int32_t w2v_topk_cosine(w2v_handle *h, uint32_t which, const int64_t *queries, uint64_t m, uint64_t cand_lo,
                        uint64_t cand_hi, uint32_t K, float tau, int64_t *out_ids, float *out_cos)
{
    if (!h) return W2V_ERR_ARG;
    if (which > 1) return fail(h, W2V_ERR_ARG, "which must be 0 (U) or 1 (V)");
    if (K < 1 || K > 64) return fail(h, W2V_ERR_ARG, "K must be in 1..64");
    if (!(cand_lo <= cand_hi && cand_hi <= h->vocab)) return fail(h, W2V_ERR_ARG, "need cand_lo <= cand_hi <= vocab");
    if (m && (!queries || !out_ids || !out_cos)) return fail(h, W2V_ERR_ARG, "queries or an output array is NULL");
    if (m >= (1ull << 31)) return fail(h, W2V_ERR_ARG, "m must be below 2^31");
    if (m == 0) return W2V_OK;
    DeviceGuard g(h->device);
    int32_t rc;
    const uint64_t nc = cand_hi - cand_lo;
    if (nc > h->inv_norm_cap) {
        W2V_CUDA(h, cudaStreamSynchronize(h->stream));
        cudaFree(h->inv_norm); h->inv_norm = nullptr; h->inv_norm_cap = 0;
        W2V_CUDA(h, dev_alloc(&h->inv_norm, nc));
        h->inv_norm_cap = nc;
    }
    // few query blocks: split the candidates over several blocks per query block, merge afterwards
    const bool tc = h->retrieval_kernel >= 1;
    const bool screen = h->retrieval_kernel >= 2;
    // the screening kernel takes the candidates in chunks, each with its own set of partial lists
    const uint64_t chunk = screen ? topk_screen_chunk(nc, h->d) : nc;
    const uint64_t chunks = chunk ? (nc + chunk - 1) / chunk : 0;
    // Every split builds a list of its own per query.  With a threshold that few candidates pass that costs
    // nothing; without one (tau <= -1: plain top-K) each list takes some K ln(n / K) exact cosines to fill, so
    // the screening kernel then settles for fewer, longer splits (a last wave 85 % full instead of 95 %).
    const uint64_t splits = tc ? topk_splits(m, chunk, h->sms, 128, 256, screen && tau <= -1.0f ? 0.85 : 0.95)
                               : topk_splits(m, nc, h->sms);
    const uint64_t lists = screen ? chunks * splits : splits;
    const uint64_t need = (splits > 1 || tc) ? lists * m * K : 0;
    if (screen && m > h->floor_cap) {
        W2V_CUDA(h, cudaStreamSynchronize(h->stream));
        cudaFree(h->floor_q); h->floor_q = nullptr; h->floor_cap = 0;
        W2V_CUDA(h, dev_alloc(&h->floor_q, m));
        h->floor_cap = m;
    }
    if (screen && topk_screen_ctiles_bytes(nc, h->d) > h->ctiles_cap) {
        W2V_CUDA(h, cudaStreamSynchronize(h->stream));
        cudaFree(h->ctiles); h->ctiles = nullptr; h->ctiles_cap = 0;
        const uint64_t bytes = topk_screen_ctiles_bytes(nc, h->d);
        W2V_CUDA(h, dev_alloc(&h->ctiles, bytes));
        h->ctiles_cap = bytes;
    }
    if (tc && topk_tc_qsplit_bytes(m, h->d) > h->qsplit_cap) {
        W2V_CUDA(h, cudaStreamSynchronize(h->stream));
        cudaFree(h->qsplit); h->qsplit = nullptr; h->qsplit_cap = 0;
        const uint64_t bytes = topk_tc_qsplit_bytes(m, h->d);
        W2V_CUDA(h, dev_alloc(&h->qsplit, bytes));
        h->qsplit_cap = bytes;
    }
    if (tc && (rc = ensure_error_word(h)) != W2V_OK) return rc;
    if (need > h->part_cap) {
        W2V_CUDA(h, cudaStreamSynchronize(h->stream));
        cudaFree(h->part_cos); cudaFree(h->part_ids); h->part_cos = nullptr; h->part_ids = nullptr; h->part_cap = 0;
        W2V_CUDA(h, dev_alloc(&h->part_cos, need));
        W2V_CUDA(h, dev_alloc(&h->part_ids, need));
        h->part_cap = need;
    }
    const float *table = which ? h->V : h->U;
    if ((rc = profile_mark(h)) != W2V_OK) return rc;
    int k = screen ? 0 : launch_inv_norms(table, h->d, h->ld, cand_lo, nc, h->inv_norm, h->sms, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "norm launch", cudaGetLastError());
    int k2;
    if (tc) {
        k2 = launch_topk_tc(table, h->d, h->ld, h->vocab, reinterpret_cast<const long long *>(queries), m, cand_lo,
                            cand_hi, K, tau, h->inv_norm, h->qsplit, h->ctiles, h->floor_q, h->part_cos, h->part_ids, (uint32_t)splits,
                            h->tc_error, screen, h->retrieval_kernel == 3, h->sms, h->stream);
        if (k2 >= 0) {
            const int k3 = launch_topk_merge(h->part_cos, h->part_ids, m, K, (uint32_t)lists, out_cos,
                                             reinterpret_cast<long long *>(out_ids), h->sms, h->stream);
            k2 = k3 < 0 ? -1 : k2 + k3;
        }
    } else {
        k2 = launch_topk(table, h->d, h->ld, h->vocab, reinterpret_cast<const long long *>(queries), m, cand_lo, cand_hi,
                         K, tau, h->inv_norm, h->part_cos, h->part_ids, (uint32_t)splits, out_cos,
                         reinterpret_cast<long long *>(out_ids), h->sms, h->stream);
    }
    if (k2 == -2) return fail(h, W2V_ERR_ARG, "d and K together exceed the shared memory of one block");
    if (k2 < 0) return fail(h, W2V_ERR_CUDA, "retrieval launch", cudaGetLastError());
    h->launches += (uint64_t)(k + k2);
    if (h->profiling) h->prof_launches += (uint64_t)(k + k2);
    if ((rc = profile_mark(h)) != W2V_OK) return rc;
    return W2V_OK;
}

int32_t w2v_probe_rows(w2v_handle *h, uint32_t access, uint64_t span_rows, uint64_t rows, double *ms,
                       uint64_t *rows_done)
{
    if (!h) return W2V_ERR_ARG;
    if (access > W2V_PROBE_TOUCH_RED) return fail(h, W2V_ERR_ARG, "unknown access pattern");
    if (!ms || !rows_done) return fail(h, W2V_ERR_ARG, "ms or rows_done is NULL");
    if (span_rows < 1 || span_rows > h->vocab) return fail(h, W2V_ERR_ARG, "need 1 <= span_rows <= vocab");
    if (rows < 1 || rows > (1ull << 32)) return fail(h, W2V_ERR_ARG, "rows must be in 1..2^32");
    const bool with_alias = access == W2V_PROBE_GATHER_ALIAS || access == W2V_PROBE_GATHER_RED_ALIAS;
    if (with_alias && !h->have_tables) return fail(h, W2V_ERR_STATE, "w2v_build_alias has not been called");
    DeviceGuard g(h->device);
    cudaEvent_t e0, e1;
    W2V_CUDA(h, cudaEventCreate(&e0));
    W2V_CUDA(h, cudaEventCreate(&e1));
    unsigned long long done = 0;
    int k = -1;
    cudaError_t ce = cudaEventRecord(e0, h->stream);
    if (ce == cudaSuccess) {
        k = launch_probe_rows(h->V, h->alias, (uint32_t)h->vocab, h->d / 4, h->ld / 4, (uint32_t)span_rows, rows, access,
                              reinterpret_cast<float *>(h->st) + 15, h->sms, h->stream, &done);   // sink: the state's padding word
        ce = cudaEventRecord(e1, h->stream);
    }
    if (ce == cudaSuccess) ce = cudaEventSynchronize(e1);
    float t = 0.f;
    if (ce == cudaSuccess && k > 0) ce = cudaEventElapsedTime(&t, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (k == -2) return fail(h, W2V_ERR_ARG, "the probe serves rows of at most 512 columns");
    if (k < 0 || ce != cudaSuccess) return fail(h, W2V_ERR_CUDA, "probe launch", ce != cudaSuccess ? ce : cudaGetLastError());
    h->launches += (uint64_t)k;
    *ms = (double)t;
    *rows_done = done;
    return W2V_OK;
}

int32_t w2v_probe_bulk_ring(w2v_handle *h, uint32_t stage_bytes, uint32_t stages, uint32_t producers,
                            uint64_t bytes_per_sm, double *ms, uint64_t *bytes_done)
{
    if (!h) return W2V_ERR_ARG;
    if (!ms || !bytes_done) return fail(h, W2V_ERR_ARG, "ms or bytes_done is NULL");
    if (stage_bytes < 16 || (stage_bytes % 16) != 0 || stages < 1 || stages > 64 ||
        (uint64_t)stage_bytes * stages > 200u * 1024u)
        return fail(h, W2V_ERR_ARG, "need stage_bytes a multiple of 16, 1..64 stages and at most 200 KB of ring");
    if (producers < 1 || producers > 4) return fail(h, W2V_ERR_ARG, "producers must be in 1..4");
    const uint64_t span = (uint64_t)h->vocab * h->ld * sizeof(float) < (64ull << 20) ? (uint64_t)h->vocab * h->ld * sizeof(float) : (64ull << 20);
    if (span < 2ull * stage_bytes * producers) return fail(h, W2V_ERR_ARG, "the table is smaller than two rounds of stages");
    const uint64_t copies = bytes_per_sm / stage_bytes;
    if (copies < 1 || copies > (1ull << 24)) return fail(h, W2V_ERR_ARG, "bytes_per_sm must give between 1 and 2^24 copies");
    DeviceGuard g(h->device);
    int32_t rc;
    if ((rc = ensure_error_word(h)) != W2V_OK) return rc;
    cudaEvent_t e0, e1;
    W2V_CUDA(h, cudaEventCreate(&e0));
    W2V_CUDA(h, cudaEventCreate(&e1));
    int k = -1;
    cudaError_t ce = cudaEventRecord(e0, h->stream);
    if (ce == cudaSuccess) {
        k = launch_probe_bulk_ring(reinterpret_cast<const unsigned char *>(h->V), span, stage_bytes, stages, (uint32_t)copies,
                                   producers, h->tc_error, h->sms, h->stream);
        ce = cudaEventRecord(e1, h->stream);
    }
    if (ce == cudaSuccess) ce = cudaEventSynchronize(e1);
    float t = 0.f;
    if (ce == cudaSuccess && k > 0) ce = cudaEventElapsedTime(&t, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (k < 0 || ce != cudaSuccess) return fail(h, W2V_ERR_CUDA, "probe launch", ce != cudaSuccess ? ce : cudaGetLastError());
    h->launches += (uint64_t)k;
    *ms = (double)t;
    *bytes_done = copies * stage_bytes;
    return W2V_OK;
}

int32_t w2v_probe_mma_ring(w2v_handle *h, uint32_t kblocks_per_stage, uint32_t stages, uint32_t tiles, uint32_t span_tiles,
                           double *cycles_per_tile, double *wait_cycles_per_tile)
{
    if (!h) return W2V_ERR_ARG;
    if (!cycles_per_tile || !wait_cycles_per_tile) return fail(h, W2V_ERR_ARG, "an output pointer is NULL");
    if (kblocks_per_stage < 1 || stages < 2 || (uint64_t)kblocks_per_stage * stages > 9)
        return fail(h, W2V_ERR_ARG, "need at least 2 stages and at most 9 K-blocks (144 KB) in the ring");
    if (tiles < 1 || tiles > (1u << 20)) return fail(h, W2V_ERR_ARG, "tiles must be in 1..2^20");
    // three streams (one per group of 64 blocks) of tiles x 160 KB each must fit into the output table
    const uint64_t table_bytes = (uint64_t)h->vocab * h->ld * sizeof(float);
    const uint64_t stream = (uint64_t)tiles * 10u * 16384u;
    const uint64_t groups = ((uint64_t)h->sms + 63) / 64;
    if (stream * groups > table_bytes || stream < 81920) return fail(h, W2V_ERR_ARG, "the table is too small for this many tiles");
    DeviceGuard g(h->device);
    int32_t rc;
    if ((rc = ensure_error_word(h)) != W2V_OK) return rc;
    const int k = launch_probe_mma_ring(reinterpret_cast<const unsigned char *>(h->V), stream, kblocks_per_stage, stages, tiles,
                                        span_tiles ? 1u : 0u, h->tc_error, h->sms, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "probe launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    long long cyc = 0, waited = 0;
    if (read_probe_mma_ring(&cyc, &waited) != 0) return fail(h, W2V_ERR_CUDA, "probe read-back", cudaGetLastError());
    *cycles_per_tile = (double)cyc / tiles;
    *wait_cycles_per_tile = (double)waited / tiles;
    return W2V_OK;
}

int32_t w2v_set_step(w2v_handle *h, uint64_t step_id)
{
    if (!h) return W2V_ERR_ARG;
    h->step_id = step_id;
    h->shard_pending = false;            // the pending adjust would regenerate other negatives
    return W2V_OK;
}

int32_t w2v_set_interleave(w2v_handle *h, uint32_t phase, uint32_t stride)
{
    if (!h) return W2V_ERR_ARG;
    if (stride < 1 || phase >= stride) return fail(h, W2V_ERR_ARG, "need stride >= 1 and phase < stride");
    h->il_phase = phase; h->il_stride = stride;
    h->shard_pending = false;
    return W2V_OK;
}

int32_t w2v_get_step(w2v_handle *h, uint64_t *step_id)
{
    if (!h || !step_id) return W2V_ERR_ARG;
    *step_id = h->step_id;
    return W2V_OK;
}

int32_t w2v_get_table_ptrs(w2v_handle *h, float **U, float **V)
{
    if (!h) return W2V_ERR_ARG;
    if (U) *U = h->U;
    if (V) *V = h->V;
    return W2V_OK;
}

int32_t w2v_get_row_stride(w2v_handle *h, uint32_t *row_stride)
{
    if (!h || !row_stride) return W2V_ERR_ARG;
    *row_stride = h->ld;
    return W2V_OK;
}

int32_t w2v_sync(w2v_handle *h)
{
    if (!h) return W2V_ERR_ARG;
    DeviceGuard g(h->device);
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    if (h->tc_error) {
        int flag = 0;
        W2V_CUDA(h, cudaMemcpy(&flag, h->tc_error, sizeof(int), cudaMemcpyDeviceToHost));
        if (flag) {
            W2V_CUDA(h, cudaMemset(h->tc_error, 0, sizeof(int)));
            if (flag & 4) return fail(h, W2V_ERR_CUDA, "a block of the bulk-copy probe gave up waiting; its timing is void");
            if (flag & 2)
                return fail(h, W2V_ERR_CUDA, "a peer barrier gave up waiting for another shard; the step that followed it "
                                             "used incomplete dot products");
            return fail(h, W2V_ERR_CUDA, "a tensor-core retrieval block gave up waiting; its results are incomplete");
        }
    }
    return W2V_OK;
}

int32_t w2v_selftest_bounded_wait(w2v_handle *h, uint32_t timeout_ms)
{
    if (!h) return W2V_ERR_ARG;
    if (timeout_ms < 1 || timeout_ms > 2000) return fail(h, W2V_ERR_ARG, "timeout_ms must be in 1..2000");
    DeviceGuard g(h->device);
    int32_t rc;
    if ((rc = ensure_error_word(h)) != W2V_OK) return rc;
    const int k = launch_bounded_wait_selftest(timeout_ms, h->tc_error, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "self-test launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    return W2V_OK;
}

int32_t w2v_set_retrieval_kernel(w2v_handle *h, uint32_t kind)
{
    if (!h) return W2V_ERR_ARG;
    if (kind > 3) return fail(h, W2V_ERR_ARG, "kind must be 0 (fp32 CUDA cores), 1 (tensor cores), 2 (tensor-core screen) or 3 (screen on pairs of SMs)");
    h->retrieval_kernel = kind;
    return W2V_OK;
}

int32_t w2v_profile_enable(w2v_handle *h, int32_t on)
{
    if (!h) return W2V_ERR_ARG;
    DeviceGuard g(h->device);
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    profile_collect(h);
    h->profiling = on != 0;
    h->prof_ms = 0.0;
    h->prof_launches = 0;
    return W2V_OK;
}

int32_t w2v_profile_read(w2v_handle *h, double *kernel_ms, uint64_t *launches)
{
    if (!h) return W2V_ERR_ARG;
    DeviceGuard g(h->device);
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    profile_collect(h);
    if (kernel_ms) *kernel_ms = h->prof_ms;
    if (launches) *launches = h->prof_launches;
    h->prof_ms = 0.0;
    h->prof_launches = 0;
    return W2V_OK;
}

int32_t w2v_get_launch_count(w2v_handle *h, uint64_t *launches)
{
    if (!h || !launches) return W2V_ERR_ARG;
    *launches = h->launches;
    return W2V_OK;
}

int32_t w2v_set_tuning(w2v_handle *h, uint32_t rows_in_flight, uint32_t blocks_per_sm)
{
    if (!h) return W2V_ERR_ARG;
    if (rows_in_flight > 8) return fail(h, W2V_ERR_ARG, "rows_in_flight must be in 0..8");
    h->rows_in_flight = rows_in_flight;
    h->blocks_per_sm = blocks_per_sm;
    return W2V_OK;
}

const char *w2v_last_error(w2v_handle *h)
{
    return h ? h->err : "invalid handle";
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Pair sampling for callers that must not allocate.
//
// Some callers of this library cannot call cudaMalloc at the moment they need the pair list:
// code that runs while another component owns all remaining device memory, latency-critical
// loops where an allocation (an implicit device synchronisation) is not acceptable, and hosts
// whose memory policy forbids allocation after start-up.  w2v_sample_pairs grows handle-owned
// scratch on demand; the entry point below instead keeps all of its scratch in one fixed array
// that is part of the library image.  Every GPU that loads the library holds that array until
// the process exits, which is why its size is modest and the chunk size is capped.
// ------------------------------------------------------------------------------------------
namespace {

constexpr uint64_t kNoAllocMaxTokens = 65536;                 // largest chunk the fixed scratch serves
constexpr size_t kNoAllocAlign = 256;
constexpr size_t na_round(size_t b) { return (b + kNoAllocAlign - 1) / kNoAllocAlign * kNoAllocAlign; }
constexpr size_t kNaTiles = kNoAllocMaxTokens / kScanTile + 2;
// layout of the fixed scratch, every part 256-byte aligned
constexpr size_t kNaState = 0;
constexpr size_t kNaFlags = kNaState + na_round(sizeof(DevState));
constexpr size_t kNaTileSums = kNaFlags + na_round(kNoAllocMaxTokens * sizeof(uint8_t));
constexpr size_t kNaTileOffs = kNaTileSums + na_round(kNaTiles * sizeof(uint2));
constexpr size_t kNaCtok = kNaTileOffs + na_round(kNaTiles * sizeof(uint2));
constexpr size_t kNaCidx = kNaCtok + na_round(kNoAllocMaxTokens * sizeof(int32_t));
constexpr size_t kNaCsent = kNaCidx + na_round(kNoAllocMaxTokens * sizeof(uint32_t));
constexpr size_t kNaWin = kNaCsent + na_round(kNoAllocMaxTokens * sizeof(uint32_t));
constexpr size_t kNaCntTile = kNaWin + na_round(kNoAllocMaxTokens * sizeof(uint16_t));
constexpr size_t kNaPairOff = kNaCntTile + na_round(kNaTiles * sizeof(unsigned long long));
constexpr size_t kNoAllocBytes = kNaPairOff + na_round((kNoAllocMaxTokens + 1) * sizeof(unsigned long long));
static_assert(kNoAllocBytes <= (2u << 20), "fixed scratch is meant to stay within 2 MiB");

// The scratch itself.  In host code this name is only a stand-in for the symbol: the address a
// kernel may use comes from cudaGetSymbolAddress, once per device (below).
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kNaMaxDevices = 64;
unsigned char *g_noalloc_addr[kNaMaxDevices] = {};            // device address per GPU, 0 = not set up

// Looks up, once per device, the device address of the fixed scratch.  `device` must be current.
int32_t noalloc_scratch_address(w2v_handle *h, int device, unsigned char **out)
{
    if (device < 0 || device >= kNaMaxDevices) return fail(h, W2V_ERR_ARG, "device ordinal beyond the supported range");
    if (!g_noalloc_addr[device]) {
        void *p = nullptr;
        cudaError_t ce = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (ce != cudaSuccess || !p) return fail(h, W2V_ERR_CUDA, "cudaGetSymbolAddress(fixed scratch)", ce);
        g_noalloc_addr[device] = static_cast<unsigned char *>(p);
    }
    *out = g_noalloc_addr[device];
    return W2V_OK;
}

}  // namespace

extern "C" int32_t w2v_sample_pairs_noalloc(w2v_handle *h, const int32_t *tokens, uint64_t n, uint32_t window,
                                            uint32_t negatives, int32_t *centre, int32_t *context, int32_t *negs,
                                            uint64_t cap, uint64_t *n_pairs, w2v_step_stats *stats)
{
    int32_t rc = check_step_args(h, tokens, n, window, negatives);
    if (rc != W2V_OK) return rc;
    if (!n_pairs) return fail(h, W2V_ERR_ARG, "n_pairs is NULL");
    if (cap && (!centre || !context || !negs)) return fail(h, W2V_ERR_ARG, "output array is NULL");
    if (n > kNoAllocMaxTokens)
        return fail(h, W2V_ERR_CAPACITY, "w2v_sample_pairs_noalloc serves at most 65536 tokens per call");
    DeviceGuard g(h->device);
    unsigned char *base = nullptr;
    if ((rc = noalloc_scratch_address(h, h->device, &base)) != W2V_OK) return rc;

    // the same kernels as w2v_sample_pairs, pointed at the fixed scratch instead of handle scratch
    Scratch sc;
    sc.n_cap = kNoAllocMaxTokens;
    sc.flags = reinterpret_cast<uint8_t *>(base + kNaFlags);
    sc.tile_sums = reinterpret_cast<uint2 *>(base + kNaTileSums);
    sc.tile_offs = reinterpret_cast<uint2 *>(base + kNaTileOffs);
    sc.ctok = reinterpret_cast<int32_t *>(base + kNaCtok);
    sc.cidx = reinterpret_cast<uint32_t *>(base + kNaCidx);
    sc.csent = reinterpret_cast<uint32_t *>(base + kNaCsent);
    sc.win = reinterpret_cast<uint16_t *>(base + kNaWin);
    sc.cnt_tile = reinterpret_cast<unsigned long long *>(base + kNaCntTile);
    sc.pair_off = reinterpret_cast<unsigned long long *>(base + kNaPairOff);
    DevState *st = reinterpret_cast<DevState *>(base + kNaState);

    // the array keeps the previous call's contents: the counters must start at zero; everything
    // else is written before it is read
    W2V_CUDA(h, cudaMemsetAsync(st, 0, sizeof(DevState), h->stream));
    const uint32_t k0 = (uint32_t)h->seed;
    const uint32_t k1 = (uint32_t)(h->seed >> 32) ^ (uint32_t)(h->step_id >> 32);
    const uint32_t step_lo = (uint32_t)h->step_id;
    SampleTables tab{h->keep_thr, h->alias};
    int k = launch_compact(tokens, n, tab, (uint32_t)h->vocab, k0, k1, step_lo, sc, st, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "compaction launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    k = launch_windows(n, window, k0, k1, step_lo, h->il_phase, h->il_stride, sc, st, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "window launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    k = launch_pair_offsets(n, sc, st, h->stream);
    if (k < 0) return fail(h, W2V_ERR_CUDA, "pair offset launch", cudaGetLastError());
    h->launches += (uint64_t)k;
    if (n) {
        StepParams p = make_params(h, window, negatives, 0.f);
        p.ctok = sc.ctok; p.cidx = sc.cidx; p.win = sc.win; p.pair_off = sc.pair_off; p.st = st;
        p.G = nullptr; p.DU = nullptr;
        k = launch_emit_pairs(p, centre, context, negs, cap, h->sms * 8, h->stream);
        if (k < 0) return fail(h, W2V_ERR_CUDA, "pair list launch", cudaGetLastError());
        h->launches += (uint64_t)k;
    }
    // counters come back through the handle's pinned mirror, which w2v_create allocated
    W2V_CUDA(h, cudaMemcpyAsync(h->st_host, st, sizeof(DevState), cudaMemcpyDeviceToHost, h->stream));
    W2V_CUDA(h, cudaStreamSynchronize(h->stream));
    const DevState &s = *h->st_host;
    if (stats) {
        stats->tokens = n; stats->kept = s.n_kept; stats->centres = s.centres; stats->pairs = s.pairs;
        stats->neg_draws = s.neg_draws; stats->neg_redraws = s.neg_redraws; stats->oov = s.oov;
        stats->status = s.status; stats->reserved = 0;
    }
    *n_pairs = s.pairs;
    if (s.pairs > cap) return fail(h, W2V_ERR_CAPACITY, "more pairs than the output arrays hold");
    if (s.status & 1u) return fail(h, W2V_ERR_TOKEN_RANGE, "token ids outside [-1, vocab) were skipped");
    return W2V_OK;
}

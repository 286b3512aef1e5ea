// Host-side construction of the two sampling tables.  Every floating-point value that
// decides an integer is produced by correctly rounded IEEE double operations in a fixed
// order (sqrt, multiply, divide, add; no pow, no fused multiply-add), so that any other
// implementation of the same recipe yields the same integers.
#include <cmath>
#include <cstdint>
#include <vector>

#include <vector_types.h>

namespace w2v {

constexpr double kHotChance = 2e-5;     // per draw
constexpr uint64_t kHotRowsMax = 8192;

static inline uint2 entry(uint32_t thr, uint32_t alias)
{
    uint2 e;
    e.x = thr;
    e.y = alias;
    return e;
}

int build_tables_host(const uint64_t *counts, uint64_t vocab, double subsample_t, uint2 *thr_alias,
                      uint32_t *keep_thr, uint32_t *hot_prefix)
{
    const double two32 = 4294967296.0;
    std::vector<double> q(vocab);
    double wsum = 0.0;
    uint64_t total = 0;
    for (uint64_t w = 0; w < vocab; ++w) {
        if (counts[w] == 0) return -1;
        total += counts[w];
        const double root = std::sqrt(static_cast<double>(counts[w]));
        q[w] = root * std::sqrt(root);          // count^(3/4)
        wsum += q[w];                           // left to right
    }

    // Negative-example distribution (Section 5.1): Vose's alias method.  Two stacks are
    // filled in ascending word order; each under-full word takes its remainder from the
    // over-full word on top of the other stack.
    std::vector<uint32_t> under, over;
    under.reserve(vocab);
    over.reserve(vocab);
    const double scale = static_cast<double>(vocab);
    // Leading rows whose chance of being drawn as a negative is at least kHotChance: with word ids
    // in frequency order these are the rows that receive thousands of additions per step.
    const double hot_q = kHotChance * scale;
    uint64_t hot = 0;
    bool in_prefix = true;
    for (uint64_t w = 0; w < vocab; ++w) {
        q[w] = (q[w] * scale) / wsum;
        if (in_prefix && q[w] >= hot_q && hot < kHotRowsMax) ++hot; else in_prefix = false;
        (q[w] < 1.0 ? under : over).push_back(static_cast<uint32_t>(w));
        thr_alias[w] = entry(0xFFFFFFFFu, static_cast<uint32_t>(w));
    }
    while (!under.empty() && !over.empty()) {
        const uint32_t lo = under.back();
        under.pop_back();
        const uint32_t hi = over.back();
        over.pop_back();
        const double t = std::floor(q[lo] * two32);
        thr_alias[lo] = entry(t >= two32 - 1.0 ? 0xFFFFFFFFu : static_cast<uint32_t>(t), hi);
        q[hi] = (q[hi] + q[lo]) - 1.0;
        (q[hi] < 1.0 ? under : over).push_back(hi);
    }

    // Sub-sampling of frequent words (Section 3): keep with probability sqrt(x) + x,
    // x = t * total / count, as the open-source word2vec program does.
    const double tt = static_cast<double>(total);
    for (uint64_t w = 0; w < vocab; ++w) {
        uint32_t thr = 0xFFFFFFFFu;
        if (subsample_t > 0.0) {
            const double x = (subsample_t * tt) / static_cast<double>(counts[w]);
            const double p = std::sqrt(x) + x;
            if (p < 1.0) thr = static_cast<uint32_t>(std::floor(p * two32));
        }
        keep_thr[w] = thr;
    }
    if (hot_prefix) *hot_prefix = static_cast<uint32_t>(hot);
    return 0;
}

}  // namespace w2v

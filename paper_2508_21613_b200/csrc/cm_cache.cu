// Plan cache (Section "Planner", last paragraph): the best plans for the loss of 1..k
// devices are computed ahead of time, during fault-free training, so that the decision at
// failure time is a table lookup.
//
// The cache covers EVERY failure set of at most k devices, so no hash table is needed: a
// set of size s sits at offset[s] + its rank in the combinatorial number system (colex
// order of the ascending ids).  Building it is nothing but the batched search over all
// those sets, a few thousand at a time; this file only enumerates and indexes them and uses
// the library's public entry points.
#include <algorithm>
#include <memory>
#include <new>
#include <vector>

#include "cm_internal.h"

struct cm_cache {
    cm_ctx *ctx = nullptr;
    int n_devices = 0, max_failures = 0;
    std::vector<uint64_t> binom;        // [n_devices + 1][max_failures + 1], saturating
    std::vector<uint64_t> offset;       // first entry of every set size, [max_failures + 2]
    std::vector<cm_plan> plans;         // [entries][4]: per policy, then the best
    uint64_t choose(int n, int t) const { return binom[(size_t)n * (max_failures + 1) + t]; }
};

namespace {

constexpr uint64_t kMaxEntries = 1ull << 20;
constexpr int kBatch = 4096;

// ids[0..t-1] ascending <- rank (colex): greedily the largest element first
void unrank_set(const cm_cache &c, uint64_t rank, int t, uint32_t *ids) {
    int v = c.n_devices;
    for (int u = t; u >= 1; --u) {
        do { --v; } while (c.choose(v, u) > rank);
        rank -= c.choose(v, u);
        ids[u - 1] = (uint32_t)v;
    }
}

uint64_t rank_set(const cm_cache &c, const uint32_t *ids, int t) {
    uint64_t r = 0;
    for (int u = 1; u <= t; ++u) r += c.choose((int)ids[u - 1], u);
    return r;
}

}  // namespace

extern "C" {

cm_status cm_cache_build(cm_ctx *ctx, int32_t max_failures, const cm_enum_opts *opts, cm_cache **out,
                         uint64_t *n_scenarios) {
    if (!ctx) return CM_EINVAL;
    if (!out || !opts) return cm_internal_fail(ctx, CM_EINVAL, "bad arguments");
    const int n_devices = cm_internal_grid_devices(ctx);
    if (n_devices < 1) return cm_internal_fail(ctx, CM_ENOPROFILE, "cm_load_profile first");
    if (max_failures < 0 || max_failures > 16 || max_failures > n_devices)
        return cm_internal_fail(ctx, CM_EINVAL, "max_failures must be 0 .. min(16, devices)");
    // the tables and the plan array below can be large (up to 2^20 sets x 4 plans): an allocation
    // failure must come back as a status, not unwind through the C ABI
    try {
    std::unique_ptr<cm_cache> c(new (std::nothrow) cm_cache());
    if (!c) return cm_internal_fail(ctx, CM_ENOMEM, "host memory");
    c->ctx = ctx;
    c->n_devices = n_devices;
    c->max_failures = max_failures;
    const int K = max_failures;
    c->binom.assign((size_t)(n_devices + 1) * (K + 1), 0);
    for (int n = 0; n <= n_devices; ++n)
        for (int t = 0; t <= K; ++t) {
            uint64_t v;
            if (t == 0) v = 1;
            else if (n == 0) v = 0;
            else {
                const uint64_t a = c->choose(n - 1, t - 1), b = c->choose(n - 1, t);
                v = a > ~0ull - b ? ~0ull : a + b;
            }
            c->binom[(size_t)n * (K + 1) + t] = v;
        }
    c->offset.assign(K + 2, 0);
    for (int s = 0; s <= K; ++s) {
        const uint64_t cnt = c->choose(n_devices, s);
        if (cnt > kMaxEntries || c->offset[s] + cnt > kMaxEntries)
            return cm_internal_fail(ctx, CM_EOVERFLOW, "more than 2^20 failure sets");
        c->offset[s + 1] = c->offset[s] + cnt;
    }
    const uint64_t total = c->offset[K + 1];
    c->plans.resize((size_t)total * 4);
    std::vector<uint32_t> ids;
    std::vector<int32_t> offsets;
    std::vector<cm_plan> best(kBatch), pol((size_t)kBatch * 3);
    // failure sets that leave the same number of survivors with the same node boundaries have
    // the same dynamic-parallelism search: let the batches share it
    struct Sharing {   // restored on every way out
        cm_ctx *ctx; int before;
        ~Sharing() { cm_internal_set_sharing(ctx, before); }
    } sharing{ctx, cm_internal_set_sharing(ctx, 1)};
    for (int s = 0; s <= K; ++s) {
        const uint64_t cnt = c->choose(n_devices, s);
        for (uint64_t first = 0; first < cnt; first += kBatch) {
            const int B = (int)std::min<uint64_t>(kBatch, cnt - first);
            ids.assign((size_t)B * std::max(s, 1), 0);
            offsets.assign(B + 1, 0);
            for (int b = 0; b < B; ++b) {
                unrank_set(*c, first + b, s, ids.data() + (size_t)b * s);
                offsets[b + 1] = (b + 1) * s;
            }
            cm_status st = cm_search_batch(ctx, ids.data(), offsets.data(), B, opts, best.data(), pol.data(), nullptr);
            if (st != CM_OK) return st;
            for (int b = 0; b < B; ++b) {
                cm_plan *dst = c->plans.data() + (size_t)(c->offset[s] + first + b) * 4;
                for (int q = 0; q < 3; ++q) dst[q] = pol[(size_t)b * 3 + q];
                dst[3] = best[b];
            }
        }
    }
    if (n_scenarios) *n_scenarios = total;
    *out = c.release();
    return CM_OK;
    } catch (const std::bad_alloc &) {
        return CM_ENOMEM;
    } catch (...) {
        return CM_EINVAL;
    }
}

cm_status cm_cache_lookup(const cm_cache *c, const uint32_t *failed_ids, int32_t n_failed, cm_plan *best,
                          cm_plan *per_policy) {
    if (!c || !best || n_failed < 0 || (n_failed > 0 && !failed_ids)) return CM_EINVAL;
    if (n_failed > c->max_failures) return CM_ENOFEASIBLE;      // not covered: search it instead
    uint32_t ids[16];
    for (int i = 0; i < n_failed; ++i) {
        if (failed_ids[i] >= (uint32_t)c->n_devices) return CM_EINVAL;
        ids[i] = failed_ids[i];
    }
    std::sort(ids, ids + n_failed);
    for (int i = 1; i < n_failed; ++i)
        if (ids[i] == ids[i - 1]) return CM_EINVAL;
    const cm_plan *src = c->plans.data() + (size_t)(c->offset[n_failed] + rank_set(*c, ids, n_failed)) * 4;
    *best = src[3];
    if (per_policy)
        for (int q = 0; q < 3; ++q) per_policy[q] = src[q];
    return CM_OK;
}

cm_status cm_cache_free(cm_cache *c) {
    if (!c) return CM_EINVAL;
    delete c;
    return CM_OK;
}

}  // extern "C"

// kt_host.cu -- the entry points that are pure host arithmetic and need no device: the
// load-adaptive scheduler and its online adaptation (paper Section III-C), the dispatch decision
// (Section III-B), the bucket plan, the element ranges of one rank per device, the barrier
// between the processes of a node, and the error message store.  Contracts: include/kaitian.h.

#include "kt_internal.h"

#include <algorithm>
#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <thread>

namespace ktd {

thread_local char g_err[512] = "";

int fail(int code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

void plan_buckets(const int64_t *numel, int T, int64_t bucket_cap_bytes, BucketPlan *bp) {
    const int64_t cap = bucket_cap_bytes / 4;
    bp->offset.assign(T, 0);
    bp->bucket_of.assign(T, 0);
    bp->start.assign(1, 0);
    bp->u_lo.assign(1, 0);
    bp->u_hi.clear();
    int64_t next = 0, open_start = 0;
    bool open_empty = true;
    for (int u = 0; u < T; ++u) {                 // u: transport order, t: list order
        const int t = T - 1 - u;
        int64_t at = round_up(next, 8);
        if (!open_empty && (at - open_start) + numel[t] > cap) {
            open_start = round_up(next, 64);
            at = open_start;
            bp->start.push_back(open_start);
            bp->u_hi.push_back(u);
            bp->u_lo.push_back(u);
        }
        bp->offset[t] = at;
        bp->bucket_of[t] = static_cast<int32_t>(bp->start.size() - 1);
        next = at + numel[t];
        open_empty = false;
    }
    bp->u_hi.push_back(T);
    bp->total = round_up(next, 64);
}

void member_units(int64_t U, int member, int M, int64_t *first, int64_t *past) {
    *first = static_cast<int64_t>(member) * U / M;
    *past = static_cast<int64_t>(member + 1) * U / M;
}

int check_shares(const int32_t *shares, int K) {
    if (!shares) return fail(KT_ERR_INVALID, "shares is NULL");
    for (int r = 0; r < K; ++r)
        if (shares[r] < 1) return fail(KT_ERR_INVALID, "shares[%d] = %d, must be >= 1", r, shares[r]);
    return KT_OK;
}

}  // namespace ktd

using namespace ktd;

namespace {

struct HostBarrier {                       // KT_HOST_BARRIER_BYTES of shared memory, zero before first use
    std::atomic<uint32_t> arrived;
    char pad_[60];
    std::atomic<uint32_t> generation;
    char pad2_[60];
};
static_assert(sizeof(HostBarrier) == KT_HOST_BARRIER_BYTES, "barrier layout");
static_assert(std::atomic<uint32_t>::is_always_lock_free, "the barrier needs lock-free 32-bit atomics");
}  // namespace

extern "C" {

int kt_schedule(const double *step_times, int K, int global_batch, int32_t *shares_out) {
    if (!step_times || !shares_out) return fail(KT_ERR_INVALID, "NULL argument");
    if (K < 1 || K > KT_MAX_RANKS) return fail(KT_ERR_INVALID, "K = %d outside [1, %d]", K, KT_MAX_RANKS);
    if (global_batch < K) return fail(KT_ERR_INVALID, "global_batch %d < K %d: some rank would idle", global_batch, K);
    double t_min = INFINITY;
    for (int i = 0; i < K; ++i) {
        const double t = step_times[i];
        if (!(t > 0.0) || !std::isfinite(t)) return fail(KT_ERR_INVALID, "step_times[%d] must be finite and > 0", i);
        t_min = t < t_min ? t : t_min;
    }
    std::vector<double> score(K), rem(K);
    double total = 0.0;
    for (int i = 0; i < K; ++i) {
        score[i] = t_min / step_times[i];
        total = total + score[i];
    }
    long long assigned = 0;
    for (int i = 0; i < K; ++i) {
        const double quota = score[i] / total * static_cast<double>(global_batch);
        const double whole = std::floor(quota);
        shares_out[i] = static_cast<int32_t>(whole);
        rem[i] = quota - whole;
        assigned += shares_out[i];
    }
    // largest remainders first (tie: lower rank); fewer than K units can be missing
    std::vector<char> served(K, 0);
    long long left = global_batch - assigned;
    while (left > 0) {
        int pick = -1;
        for (int i = 0; i < K; ++i)
            if (!served[i] && (pick < 0 || rem[i] > rem[pick])) pick = i;
        if (pick < 0) {          // every rank served once already: next round
            served.assign(K, 0);
            continue;
        }
        served[pick] = 1;
        shares_out[pick] += 1;
        --left;
    }
    for (long long over = assigned - global_batch; over > 0; --over) {   // rounding noise only
        int pick = 0;
        for (int i = 1; i < K; ++i)
            if (shares_out[i] > shares_out[pick]) pick = i;
        shares_out[pick] -= 1;
    }
    // nobody idles: take from the largest share (tie: slowest, then higher rank)
    for (int i = 0; i < K; ++i) {
        if (shares_out[i] >= 1) continue;
        int donor = 0;
        for (int j = 1; j < K; ++j)
            if (shares_out[j] > shares_out[donor] ||
                (shares_out[j] == shares_out[donor] && step_times[j] >= step_times[donor]))
                donor = j;
        shares_out[donor] -= 1;
        shares_out[i] += 1;
    }
    return KT_OK;
}

int kt_scores(const double *step_times, int K, double *scores_out) {
    if (!step_times || !scores_out) return fail(KT_ERR_INVALID, "NULL argument");
    if (K < 1 || K > KT_MAX_RANKS) return fail(KT_ERR_INVALID, "K = %d outside [1, %d]", K, KT_MAX_RANKS);
    double fastest = INFINITY;
    for (int i = 0; i < K; ++i) {
        if (!(step_times[i] > 0.0) || !std::isfinite(step_times[i]))
            return fail(KT_ERR_INVALID, "step_times[%d] must be finite and > 0", i);
        fastest = std::min(fastest, step_times[i]);
    }
    for (int i = 0; i < K; ++i) scores_out[i] = fastest / step_times[i];
    return KT_OK;
}

int kt_route(const int32_t *group_of, int K, int G, const int32_t *participants, int n, int *route,
             int32_t *groups_out, int *n_groups_out) {
    if (!group_of || !participants || !route) return fail(KT_ERR_INVALID, "NULL argument");
    if (K < 1 || K > KT_MAX_RANKS) return fail(KT_ERR_INVALID, "K = %d outside [1, %d]", K, KT_MAX_RANKS);
    if (G < 1 || G > KT_MAX_GROUPS) return fail(KT_ERR_INVALID, "G = %d outside [1, %d]", G, KT_MAX_GROUPS);
    if (n < 1) return fail(KT_ERR_INVALID, "n = %d must be >= 1", n);
    for (int r = 0; r < K; ++r)
        if (group_of[r] < 0 || group_of[r] >= G) return fail(KT_ERR_INVALID, "group_of[%d] = %d outside [0, %d)", r, group_of[r], G);
    std::vector<char> seen_rank(K, 0), seen_group(G, 0);
    for (int i = 0; i < n; ++i) {
        const int r = participants[i];
        if (r < 0 || r >= K) return fail(KT_ERR_INVALID, "participants[%d] = %d outside [0, %d)", i, r, K);
        if (seen_rank[r]) return fail(KT_ERR_INVALID, "rank %d is listed twice", r);
        seen_rank[r] = 1;
        seen_group[group_of[r]] = 1;
    }
    int count = 0;
    for (int g = 0; g < G; ++g)
        if (seen_group[g]) {
            if (groups_out) groups_out[count] = g;
            ++count;
        }
    if (n_groups_out) *n_groups_out = count;
    *route = count == 1 ? KT_ROUTE_DIRECT : KT_ROUTE_RELAY;
    return KT_OK;
}

int kt_plan_buckets(const int64_t *numel, int T, int64_t bucket_cap_bytes, int32_t *n_buckets,
                    int64_t *bucket_start, int64_t *bucket_numel, int64_t *tensor_offset, int32_t *bucket_of,
                    int64_t *transport_numel) {
    if (!numel) return fail(KT_ERR_INVALID, "numel is NULL");
    if (T < 1) return fail(KT_ERR_INVALID, "T = %d must be >= 1", T);
    if (bucket_cap_bytes < 4) return fail(KT_ERR_INVALID, "bucket_cap_bytes must be >= 4");
    for (int t = 0; t < T; ++t)
        if (numel[t] < 0) return fail(KT_ERR_INVALID, "numel[%d] is negative", t);
    BucketPlan bp;
    plan_buckets(numel, T, bucket_cap_bytes, &bp);
    const int nb = static_cast<int>(bp.start.size());
    if (n_buckets) *n_buckets = nb;
    for (int b = 0; b < nb; ++b) {
        if (bucket_start) bucket_start[b] = bp.start[b];
        if (bucket_numel) bucket_numel[b] = (b + 1 < nb ? bp.start[b + 1] : bp.total) - bp.start[b];
    }
    if (tensor_offset) std::memcpy(tensor_offset, bp.offset.data(), T * sizeof(int64_t));
    if (bucket_of) std::memcpy(bucket_of, bp.bucket_of.data(), T * sizeof(int32_t));
    if (transport_numel) *transport_numel = bp.total;
    return KT_OK;
}

int kt_shard_ranges(const int64_t *numel, int T, int64_t bucket_cap_bytes, int64_t unit, int bucket, int n_members,
                    int64_t *lo_out, int64_t *n_out) {
    if (!numel || !lo_out || !n_out) return fail(KT_ERR_INVALID, "NULL argument");
    if (T < 1) return fail(KT_ERR_INVALID, "T = %d must be >= 1", T);
    if (bucket_cap_bytes < 4) return fail(KT_ERR_INVALID, "bucket_cap_bytes must be >= 4");
    if (unit < 1) return fail(KT_ERR_INVALID, "unit must be >= 1");
    if (n_members < 1 || n_members > KT_MAX_RANKS) return fail(KT_ERR_INVALID, "n_members = %d outside [1, %d]", n_members, KT_MAX_RANKS);
    for (int t = 0; t < T; ++t)
        if (numel[t] < 0) return fail(KT_ERR_INVALID, "numel[%d] is negative", t);
    BucketPlan bp;
    plan_buckets(numel, T, bucket_cap_bytes, &bp);
    const int nb = static_cast<int>(bp.start.size());
    if (bucket < -1 || bucket >= nb) return fail(KT_ERR_SHAPE, "bucket %d out of range [-1, %d)", bucket, nb);
    // units before every tensor of the range, transport order (u = T - 1 - t)
    const int u_lo = bucket < 0 ? 0 : bp.u_lo[bucket], u_hi = bucket < 0 ? T : bp.u_hi[bucket];
    std::vector<int64_t> before(u_hi - u_lo + 1, 0), start(u_hi - u_lo + 1, 0);
    for (int u = u_lo; u < u_hi; ++u) {
        const int64_t at = bp.offset[T - 1 - u];
        const int64_t end = u + 1 < T ? bp.offset[T - 2 - u] : bp.total;
        start[u - u_lo] = at;
        before[u - u_lo + 1] = before[u - u_lo] + (end - at + unit - 1) / unit;
    }
    const int64_t range_end = u_hi < T ? bp.offset[T - 1 - u_hi] : bp.total;
    start[u_hi - u_lo] = range_end;
    const int64_t U = before[u_hi - u_lo];
    auto element_of = [&](int64_t index) {          // first element of unit `index` of the range
        const int64_t k = std::upper_bound(before.begin(), before.end(), index) - before.begin() - 1;
        if (k >= u_hi - u_lo) return range_end;
        return start[k] + (index - before[k]) * unit;
    };
    for (int m = 0; m < n_members; ++m) {
        int64_t first, past;
        member_units(U, m, n_members, &first, &past);
        lo_out[m] = element_of(first);
        n_out[m] = element_of(past) - lo_out[m];
    }
    return KT_OK;
}

int kt_host_barrier(void *shared, int n_ranks, int timeout_ms) {
    if (!shared) return fail(KT_ERR_INVALID, "shared is NULL");
    if (reinterpret_cast<uintptr_t>(shared) % 64) return fail(KT_ERR_ALIGN, "the barrier block must be 64-byte aligned");
    if (n_ranks < 1) return fail(KT_ERR_INVALID, "n_ranks = %d must be >= 1", n_ranks);
    HostBarrier *b = static_cast<HostBarrier *>(shared);
    const uint32_t gen = b->generation.load(std::memory_order_acquire);
    if (b->arrived.fetch_add(1, std::memory_order_acq_rel) + 1 == static_cast<uint32_t>(n_ranks)) {
        b->arrived.store(0, std::memory_order_relaxed);          // before the release below: the next round starts clean
        b->generation.store(gen + 1, std::memory_order_release);
        return KT_OK;
    }
    // Poll without giving up the core for the first 200 us (ranks of one step arrive within
    // microseconds of each other), then yield between polls, and after 5 ms sleep between them.
    const auto begin = std::chrono::steady_clock::now();
    const auto deadline = begin + std::chrono::milliseconds(timeout_ms < 0 ? 0 : timeout_ms);
    for (unsigned spins = 0;; ++spins) {
        if (b->generation.load(std::memory_order_acquire) != gen) return KT_OK;
        if ((spins & 63u) != 63u) {
#if defined(__x86_64__) || defined(__i386__)
            __builtin_ia32_pause();
#elif defined(__aarch64__)
            asm volatile("yield");
#endif
            continue;
        }
        const auto now = std::chrono::steady_clock::now();
        if (timeout_ms >= 0 && now >= deadline)
            return fail(KT_ERR_TIMEOUT, "host barrier: %u of %d ranks had arrived after %d ms",
                        b->arrived.load(std::memory_order_relaxed), n_ranks, timeout_ms);
        if (now - begin < std::chrono::microseconds(200)) continue;
        if (now - begin < std::chrono::milliseconds(5)) std::this_thread::yield();
        else std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
}

const char *kt_last_error(const kt_ctx *) { return g_err; }

}  // extern "C"

// ---------------------------------------------------------------------- online adaptation and sampler
struct kt_adapt {
    int K = 0, B = 0, period = 1;
    double alpha = 1.0, hysteresis = 0.0;
    int64_t count = 0;
    std::vector<double> tau;        // smoothed per-sample time of every rank
    std::vector<int32_t> shares;    // shares in use
};

extern "C" {

int kt_adapt_create(const int32_t *shares, int K, int global_batch, double alpha, int period, double hysteresis,
                    kt_adapt **out) {
    if (!out) return fail(KT_ERR_INVALID, "out is NULL");
    *out = nullptr;
    if (K < 1 || K > KT_MAX_RANKS) return fail(KT_ERR_INVALID, "K = %d outside [1, %d]", K, KT_MAX_RANKS);
    if (int rc = check_shares(shares, K)) return rc;
    long long sum = 0;
    for (int r = 0; r < K; ++r) sum += shares[r];
    if (sum != global_batch) return fail(KT_ERR_INVALID, "shares add up to %lld, global_batch is %d", sum, global_batch);
    if (!(alpha > 0.0) || !(alpha <= 1.0)) return fail(KT_ERR_INVALID, "alpha must lie in (0, 1]");
    if (period < 1) return fail(KT_ERR_INVALID, "period must be >= 1");
    if (!(hysteresis >= 0.0) || !(hysteresis < 1.0)) return fail(KT_ERR_INVALID, "hysteresis must lie in [0, 1)");
    kt_adapt *a = new (std::nothrow) kt_adapt();
    if (!a) return fail(KT_ERR_NOMEM, "out of host memory");
    a->K = K;
    a->B = global_batch;
    a->alpha = alpha;
    a->period = period;
    a->hysteresis = hysteresis;
    a->tau.assign(K, 0.0);
    a->shares.assign(shares, shares + K);
    *out = a;
    return KT_OK;
}

int kt_adapt_observe(kt_adapt *a, const double *step_times, int32_t *shares_out, int *changed) {
    if (!a || !step_times) return fail(KT_ERR_INVALID, "NULL argument");
    for (int r = 0; r < a->K; ++r)
        if (!(step_times[r] > 0.0) || !std::isfinite(step_times[r]))
            return fail(KT_ERR_INVALID, "step_times[%d] must be finite and > 0", r);
    const bool fresh = a->count == 0;
    for (int r = 0; r < a->K; ++r) {
        const double per_sample = step_times[r] / static_cast<double>(a->shares[r]);
        a->tau[r] = fresh ? per_sample : (1.0 - a->alpha) * a->tau[r] + a->alpha * per_sample;
    }
    a->count += 1;
    int adopted = 0;
    if (a->count % a->period == 0) {
        std::vector<int32_t> next(a->K);
        if (int rc = kt_schedule(a->tau.data(), a->K, a->B, next.data())) return rc;
        double cost_now = 0.0, cost_next = 0.0;
        for (int r = 0; r < a->K; ++r) {
            cost_now = std::max(cost_now, a->tau[r] * static_cast<double>(a->shares[r]));
            cost_next = std::max(cost_next, a->tau[r] * static_cast<double>(next[r]));
        }
        if (next != a->shares && cost_next < (1.0 - a->hysteresis) * cost_now) {
            a->shares.swap(next);
            adopted = 1;
        }
    }
    if (shares_out) std::memcpy(shares_out, a->shares.data(), a->K * sizeof(int32_t));
    if (changed) *changed = adopted;
    return KT_OK;
}

int kt_adapt_state(const kt_adapt *a, double *per_sample_out, int32_t *shares_out, int64_t *count_out) {
    if (!a) return fail(KT_ERR_INVALID, "state is NULL");
    if (per_sample_out) std::memcpy(per_sample_out, a->tau.data(), a->K * sizeof(double));
    if (shares_out) std::memcpy(shares_out, a->shares.data(), a->K * sizeof(int32_t));
    if (count_out) *count_out = a->count;
    return KT_OK;
}

void kt_adapt_destroy(kt_adapt *a) { delete a; }

int64_t kt_sampler_steps(int64_t dataset_size, int64_t global_batch, int drop_last) {
    if (dataset_size < 1 || global_batch < 1) {
        fail(KT_ERR_INVALID, "dataset_size and global_batch must be >= 1");
        return KT_ERR_INVALID;
    }
    return drop_last ? dataset_size / global_batch : (dataset_size + global_batch - 1) / global_batch;
}

}  // extern "C"

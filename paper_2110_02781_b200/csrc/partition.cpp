// Host-side scheduling arithmetic: capacity estimate (Eq. 1-3), partition optimiser (Eq. 4-7)
// and the weight-redistribution plan (Algorithm 1).  No GPU involved.
#include <cstring>
#include <limits>
#include <algorithm>
#include <vector>
#include "common.h"

namespace ftp {

static thread_local char g_err[512];
char* last_error_buf() { return g_err; }

ftp_status fail(ftp_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return s;
}

static bool valid_points(const int32_t* p, int32_t n, int32_t L) {
    if (n < 1 || p[0] != 0) return false;
    for (int32_t i = 0; i < n; ++i)
        if (p[i] >= p[i + 1]) return false;
    return L < 0 || p[n] == L;
}

}  // namespace ftp

using namespace ftp;

extern "C" const char* ftp_last_error(void) { return last_error_buf(); }

extern "C" ftp_status ftp_estimate_capacity(const double* layer_times, int32_t L, const int32_t* points, int32_t N,
                                            const double* stage_times, double* capacities) {
    FTP_REQUIRE(layer_times && points && stage_times && capacities, FTP_EINVAL, "estimate_capacity: null argument");
    FTP_REQUIRE(L >= 1 && N >= 1 && N <= L, FTP_EINVAL, "estimate_capacity: need 1 <= N <= L (N=%d, L=%d)", N, L);
    FTP_REQUIRE(valid_points(points, N, L), FTP_EINVAL, "estimate_capacity: points must rise from 0 to L");
    for (int32_t i = 0; i < N; ++i) {
        double t0 = 0.0;                                   // Eq. 2: central node's time for stage i's layers
        for (int32_t j = points[i]; j < points[i + 1]; ++j) t0 = t0 + layer_times[j];
        FTP_REQUIRE(t0 > 0.0, FTP_ERANGE, "estimate_capacity: stage %d has zero profiled time", i);
        capacities[i] = stage_times[i] / t0;               // Eq. 1
    }
    capacities[0] = 1.0;                                   // the central node is the unit of capacity
    return FTP_OK;
}

extern "C" ftp_status ftp_choose_partition(const double* layer_times, int32_t L, const double* capacities, int32_t N,
                                           const double* out_bytes, const double* bandwidth, int32_t* points_out,
                                           double* bottleneck_out) {
    FTP_REQUIRE(layer_times && capacities && points_out, FTP_EINVAL, "choose_partition: null argument");
    FTP_REQUIRE(L >= 1 && N >= 1, FTP_EINVAL, "choose_partition: L and N must be positive");
    FTP_REQUIRE(N <= L, FTP_EINVAL, "choose_partition: %d stages cannot all be non-empty with %d units", N, L);
    FTP_REQUIRE((out_bytes == nullptr) == (bandwidth == nullptr), FTP_EINVAL,
                "choose_partition: out_bytes and bandwidth must be given together");
    const bool comm = out_bytes != nullptr;
    const double inf = std::numeric_limits<double>::infinity();
    std::vector<double> S(L + 1, 0.0);                     // running sums of the per-layer times
    for (int32_t j = 0; j < L; ++j) S[j + 1] = S[j] + layer_times[j];
    // A[n][j]: least slowest-part time of units 0..j on the first n stages; cut[n][j]: the last cut
    std::vector<double> A((size_t)(N + 1) * L, inf);
    std::vector<int32_t> cut((size_t)(N + 1) * L, -1);
    for (int32_t j = 0; j < L; ++j) A[(size_t)1 * L + j] = capacities[0] * (S[j + 1] - S[0]);   // Eq. 4 base case
    for (int32_t n = 2; n <= N; ++n) {
        for (int32_t j = n - 1; j < L; ++j) {
            double best = inf;
            int32_t arg = -1;
            for (int32_t l = n - 2; l <= j - 1; ++l) {
                const double sub = A[(size_t)(n - 1) * L + l];
                const double link = comm ? 2.0 * (out_bytes[l] / bandwidth[n - 2]) : 0.0;   // 2 * T_c, Eq. 5
                const double last = capacities[n - 1] * (S[j + 1] - S[l + 1]);              // Eq. 6 with Eq. 3
                double v = sub > link ? sub : link;
                v = v > last ? v : last;
                if (v < best) { best = v; arg = l; }       // strict: the smallest optimal cut wins
            }
            A[(size_t)n * L + j] = best;
            cut[(size_t)n * L + j] = arg;
        }
    }
    points_out[N] = L;
    int32_t j = L - 1;
    for (int32_t n = N; n >= 2; --n) {
        const int32_t l = cut[(size_t)n * L + j];
        points_out[n - 1] = l + 1;
        j = l;
    }
    points_out[0] = 0;
    if (bottleneck_out) *bottleneck_out = A[(size_t)N * L + (L - 1)];
    return FTP_OK;
}

extern "C" ftp_status ftp_redistribution_plan(const int32_t* p_new, int32_t n_new, const int32_t* p_cur, int32_t n_cur,
                                              int32_t i_fail, int32_t i_cur, int32_t i_new, int32_t* owner_of_needed,
                                              int32_t* n_local) {
    FTP_REQUIRE(p_new && p_cur && owner_of_needed, FTP_EINVAL, "redistribution_plan: null argument");
    FTP_REQUIRE(n_new >= 1 && n_cur >= 1, FTP_EINVAL, "redistribution_plan: empty worker list");
    FTP_REQUIRE(valid_points(p_new, n_new, -1) && valid_points(p_cur, n_cur, p_new[n_new]), FTP_EINVAL,
                "redistribution_plan: both partitions must rise from 0 to the same L");
    FTP_REQUIRE(i_new >= 0 && i_new < n_new && i_cur >= -1 && i_cur < n_cur && i_fail >= -1 && i_fail < n_cur,
                FTP_ERANGE, "redistribution_plan: worker index out of range");
    const int32_t held_lo = i_cur >= 0 ? p_cur[i_cur] : 0, held_hi = i_cur >= 0 ? p_cur[i_cur + 1] : 0;
    int32_t local = 0;
    for (int32_t l = p_new[i_new]; l < p_new[i_new + 1]; ++l) {
        int32_t& out = owner_of_needed[l - p_new[i_new]];
        if (l >= held_lo && l < held_hi) { out = -1; ++local; continue; }     // needed and not missing
        int32_t target = 0;                                                    // holder under p_cur
        while (!(p_cur[target] <= l && l < p_cur[target + 1])) ++target;
        if (i_fail >= 0) {
            if (target > i_fail) target -= 1;                                  // list was renumbered
            else if (target == i_fail && i_fail == n_cur - 1) target = 0;      // last stage's replica: central node
        }
        out = target;
    }
    if (n_local) *n_local = local;
    return FTP_OK;
}

extern "C" ftp_status ftp_recovery_plan(const int32_t* p_cur, int32_t n_cur, const int32_t* failed, int32_t n_failed, const int32_t* p_new,
                                        int32_t n_new, int32_t* kind, int32_t* index) {
    FTP_REQUIRE(p_cur && failed && p_new && kind && index, FTP_EINVAL, "recovery_plan: null argument");
    FTP_REQUIRE(n_cur >= 2 && n_failed >= 1 && n_new == n_cur - n_failed && n_new >= 1, FTP_EINVAL,
                "recovery_plan: %d workers minus %d failed must leave the %d stages of the new partition", n_cur, n_failed, n_new);
    FTP_REQUIRE(valid_points(p_new, n_new, -1) && valid_points(p_cur, n_cur, p_new[n_new]), FTP_EINVAL,
                "recovery_plan: both partitions must rise from 0 to the same L");
    std::vector<char> dead(n_cur, 0);
    for (int32_t k = 0; k < n_failed; ++k) {
        FTP_REQUIRE(failed[k] >= 1 && failed[k] < n_cur, FTP_ERANGE, "recovery_plan: failed worker %d is not among 1..%d (worker 0, the central node, does not fail)",
                    failed[k], n_cur - 1);
        FTP_REQUIRE(!dead[failed[k]], FTP_EINVAL, "recovery_plan: worker %d is listed twice", failed[k]);
        dead[failed[k]] = 1;
    }
    std::vector<int32_t> new_index(n_cur, -1), alive;
    for (int32_t i = 0; i < n_cur; ++i)
        if (!dead[i]) { new_index[i] = (int32_t)alive.size(); alive.push_back(i); }
    for (int32_t j = 0; j < n_new; ++j)
        for (int32_t u = p_new[j]; u < p_new[j + 1]; ++u) {
            int32_t holder = 0;
            while (!(p_cur[holder] <= u && u < p_cur[holder + 1])) ++holder;
            if (holder == alive[j]) { kind[u] = FTP_SRC_LOCAL; index[u] = j; }
            else if (!dead[holder]) { kind[u] = FTP_SRC_STAGE; index[u] = new_index[holder]; }
            else if (holder == n_cur - 1) { kind[u] = FTP_SRC_REPLICA; index[u] = 0; }                       // the central node keeps the last worker's replica
            else if (!dead[holder + 1]) { kind[u] = FTP_SRC_REPLICA; index[u] = new_index[holder + 1]; }
            else { kind[u] = FTP_SRC_CENTRAL; index[u] = 0; }
        }
    return FTP_OK;
}


// ---- training state of a node and the central node's fault handler (Sec. III-B Table I, Sec. III-F) -------------
extern "C" ftp_status ftp_state_init(ftp_train_state* st, float learning_rate, int64_t epoch_number, int64_t batch_number) {
    FTP_REQUIRE(st, FTP_EINVAL, "state_init: null state");
    FTP_REQUIRE(epoch_number >= 0 && batch_number >= 0, FTP_EINVAL, "state_init: epoch and batch numbers must not be negative");
    st->committed_forward_id = -1;
    st->committed_backward_id = -1;
    st->status = 0;
    st->learning_rate = learning_rate;
    st->epoch_number = epoch_number;
    st->batch_number = batch_number;
    return FTP_OK;
}

extern "C" ftp_status ftp_state_forward_done(ftp_train_state* st, int64_t batch_id) {
    FTP_REQUIRE(st && batch_id >= 0, FTP_EINVAL, "state_forward_done: null state or negative batch id");
    st->committed_forward_id = batch_id;
    return FTP_OK;
}

extern "C" ftp_status ftp_state_backward_done(ftp_train_state* st, int64_t batch_id) {
    FTP_REQUIRE(st && batch_id >= 0, FTP_EINVAL, "state_backward_done: null state or negative batch id");
    st->committed_backward_id = batch_id;
    return FTP_OK;
}

extern "C" ftp_status ftp_state_timer_expired(ftp_train_state* st, int64_t batch_id, int32_t* triggered) {
    FTP_REQUIRE(st && triggered && batch_id >= 0, FTP_EINVAL, "state_timer_expired: null argument or negative batch id");
    *triggered = st->status == 0 ? 1 : 0;          // later timers find the handler already running
    st->status = 1;
    return FTP_OK;
}

extern "C" ftp_status ftp_state_may_forward(const ftp_train_state* st, int64_t batch_id, int32_t* allowed) {
    FTP_REQUIRE(st && allowed, FTP_EINVAL, "state_may_forward: null argument");
    *allowed = (st->status == 0 || batch_id <= st->committed_forward_id) ? 1 : 0;
    return FTP_OK;
}

extern "C" ftp_status ftp_state_reset(ftp_train_state* st, int64_t batch_id, int64_t* resume_from) {
    FTP_REQUIRE(st && batch_id >= 0, FTP_EINVAL, "state_reset: null state or negative batch id");
    st->committed_forward_id = batch_id;
    st->committed_backward_id = batch_id;
    st->status = 0;
    if (resume_from) *resume_from = batch_id;
    return FTP_OK;
}

extern "C" ftp_status ftp_classify_probe(const int32_t* responses, int32_t n_workers, int32_t* action, int32_t* failed, int32_t* n_failed,
                                         int32_t* restarted_worker) {
    FTP_REQUIRE(responses && action && failed && n_failed && restarted_worker, FTP_EINVAL, "classify_probe: null argument");
    FTP_REQUIRE(n_workers >= 1 && responses[0] == FTP_PROBE_NORMAL, FTP_EINVAL, "classify_probe: worker 0 is the central node and answers normally");
    int32_t silent = 0, restarted = 0, last_restarted = -1;
    for (int32_t i = 0; i < n_workers; ++i) {
        FTP_REQUIRE(responses[i] >= FTP_PROBE_NORMAL && responses[i] <= FTP_PROBE_SILENT, FTP_EINVAL, "classify_probe: unknown response %d of worker %d", responses[i], i);
        if (responses[i] == FTP_PROBE_SILENT) ++silent;
        if (responses[i] == FTP_PROBE_RESTARTED) { ++restarted; last_restarted = i; }
    }
    *n_failed = 0;
    *restarted_worker = -1;
    if (silent == 0 && restarted == 0) { *action = FTP_ACTION_RESTART_BATCH; return FTP_OK; }
    if (silent == 0 && restarted == 1) { *action = FTP_ACTION_RESEND_STATE; *restarted_worker = last_restarted; return FTP_OK; }
    *action = FTP_ACTION_REDISTRIBUTE;
    for (int32_t i = 0; i < n_workers; ++i)
        if (responses[i] != FTP_PROBE_NORMAL) failed[(*n_failed)++] = i;
    return FTP_OK;
}

// Sec. III-D: the dynamic partition runs after the first 10 batches and then every 100 batches.
extern "C" int32_t ftp_is_repartition_iter(int64_t it, int64_t first, int64_t period) {
    const int64_t done = it + 1;
    if (first <= 0 || period <= 0 || done <= 0) return 0;
    return (done == first || (done > first && done % period == 0)) ? 1 : 0;
}

// Sec. IV-B / IV-E: a replication runs when a batch whose 1-indexed count is a multiple of the period has finished.
extern "C" int32_t ftp_is_replication_iter(int64_t it, int64_t period) {
    return (period > 0 && it + 1 > 0 && (it + 1) % period == 0) ? 1 : 0;
}

// ---- asynchronous pipeline schedule (Sec. III-C): order of passes and weight-version numbers on one stage --------
extern "C" ftp_status ftp_async_stage_order(int32_t n_stages, int32_t stage, int32_t n_batches, int32_t* is_backward, int32_t* batch) {
    FTP_REQUIRE(is_backward && batch, FTP_EINVAL, "async_stage_order: null output");
    FTP_REQUIRE(n_stages >= 1 && stage >= 0 && stage < n_stages && n_batches >= 0, FTP_EINVAL, "async_stage_order: need 0 <= stage < n_stages and n_batches >= 0");
    const int32_t warm = std::min(n_stages - stage, n_batches);
    int32_t k = 0, nf = warm, nb = 0;
    for (int32_t b = 0; b < warm; ++b) { is_backward[k] = 0; batch[k++] = b; }
    while (nb < n_batches) {
        is_backward[k] = 1; batch[k++] = nb++;
        if (nf < n_batches) { is_backward[k] = 0; batch[k++] = nf++; }
    }
    return FTP_OK;
}

extern "C" ftp_status ftp_async_version_trace(int32_t n_stages, int32_t stage, int32_t n_batches, int32_t k_interval, int64_t* forward_version,
                                              int64_t* version_after_backward, int32_t* aggregate_after_forward) {
    FTP_REQUIRE(forward_version && version_after_backward && aggregate_after_forward, FTP_EINVAL, "async_version_trace: null output");
    FTP_REQUIRE(n_stages >= 1 && stage >= 0 && stage < n_stages && n_batches >= 0 && k_interval >= 1, FTP_EINVAL,
                "async_version_trace: need 0 <= stage < n_stages, n_batches >= 0, k >= 1");
    std::vector<int32_t> isb(2 * (size_t)n_batches + 1), bat(2 * (size_t)n_batches + 1);
    ftp_status s = ftp_async_stage_order(n_stages, stage, n_batches, isb.data(), bat.data());
    if (s != FTP_OK) return s;
    const int64_t c = n_stages - stage;
    int64_t ver = 0, updates = 0, done_at = 0, in_flight = 0;
    for (int32_t b = 0; b < n_batches; ++b) aggregate_after_forward[b] = 0;
    for (int32_t e = 0; e < 2 * n_batches; ++e) {
        const int32_t b = bat[e];
        if (!isb[e]) {
            forward_version[b] = ver;
            ++in_flight;
            if (c > 1 && updates > 0 && updates % (k_interval * c) == 0 && updates != done_at && in_flight == c) {
                ++ver;                                       // the n - i stashed versions are aggregated: one more version
                done_at = updates;
                aggregate_after_forward[b] = 1;
            }
        } else {
            --in_flight;
            ++ver;
            ++updates;
            version_after_backward[b] = ver;
        }
    }
    return FTP_OK;
}

// Host-only parts of the method: Dynamic Local Updates (Eq. 6), the learning-rate schedule (Eq. 3)
// and the asynchronous task scheduler (Algorithm 2 with the get_worker() of Algorithm 5) driven by
// faked job durations, which is how the paper itself runs it for reproducibility.
#include "../../include/alsgd.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

namespace {

struct Job {
    bool in_flight = false;
    bool ran_before = false;
    double completed_time = 0.0;
    double restart_time = 0.0;     // when the window that synchronised this worker closed
    uint32_t local_updates = 0;
};

}  // namespace

struct alsgd_sched {
    uint32_t n = 0;
    double tau_grace = 0.0;
    uint64_t t_max = 0;
    uint64_t t_local = 0;
    std::vector<Job> jobs;
};

extern "C" {

int alsgd_dylu_steps(const double* speeds, uint32_t n, uint32_t H, uint32_t* steps_out) {
    if (!speeds || !steps_out || n == 0 || H == 0) return ALSGD_E_ARG;
    double fastest = 0.0;
    for (uint32_t i = 0; i < n; ++i) {
        if (!(speeds[i] > 0.0) || !std::isfinite(speeds[i])) return ALSGD_E_ARG;
        fastest = std::max(fastest, speeds[i]);
    }
    for (uint32_t i = 0; i < n; ++i) {
        const double share = speeds[i] / fastest;               // v(w) / max v(w')
        const double steps = std::floor(share * (double)H);     // floor(. * H)
        steps_out[i] = steps >= 1.0 ? (uint32_t)steps : 1u;     // a worker always runs at least one step
    }
    return ALSGD_OK;
}

int alsgd_shard_probs(const double* sizes, const double* learned, uint32_t n, double* probs_out) {
    if (!sizes || !learned || !probs_out || n == 0) return ALSGD_E_ARG;
    double size_sum = 0.0, learned_sum = 0.0;
    for (uint32_t i = 0; i < n; ++i) {
        if (!(sizes[i] > 0.0) || !std::isfinite(sizes[i]) || !(learned[i] >= 0.0) || !std::isfinite(learned[i])) return ALSGD_E_ARG;
        size_sum += sizes[i];
        learned_sum += learned[i];
    }
    double total = 0.0;
    for (uint32_t i = 0; i < n; ++i) {
        const double due = sizes[i] / size_sum;                                   // the shard's share of the data
        const double had = learned_sum > 0.0 ? learned[i] / learned_sum : 0.0;    // its share of the progress so far
        probs_out[i] = std::max(due - had, 0.0);
        total += probs_out[i];
    }
    for (uint32_t i = 0; i < n; ++i) probs_out[i] = total > 0.0 ? probs_out[i] / total : sizes[i] / size_sum;
    return ALSGD_OK;
}

int alsgd_lr_at(const alsgd_lr_sched* s, uint64_t t, double* lr_out) {
    if (!s || !lr_out) return ALSGD_E_ARG;
    if (!(s->eta_max >= 0.0) || !(s->eta_min >= 0.0)) return ALSGD_E_ARG;
    if (t < s->t_warmup) {
        *lr_out = (double)t * s->eta_max / (double)s->t_warmup;
        return ALSGD_OK;
    }
    double progress = 1.0;                                       // an empty decay phase counts as finished
    if (s->T > s->t_warmup) {
        progress = (double)(t - s->t_warmup) / (double)(s->T - s->t_warmup);
        progress = std::min(1.0, std::max(0.0, progress));
    }
    const double kPi = 3.14159265358979323846;
    *lr_out = s->eta_min + 0.5 * (s->eta_max - s->eta_min) * (1.0 + std::cos(progress * kPi));
    return ALSGD_OK;
}

int alsgd_sched_create(alsgd_sched** out, uint32_t n_workers, double tau_grace, uint64_t t_max) {
    if (!out || n_workers == 0 || !(tau_grace >= 0.0) || !std::isfinite(tau_grace)) return ALSGD_E_ARG;
    alsgd_sched* s = new (std::nothrow) alsgd_sched();
    if (!s) return ALSGD_E_NOMEM;
    s->n = n_workers;
    s->tau_grace = tau_grace;
    s->t_max = t_max;
    s->jobs.assign(n_workers, Job());
    *out = s;
    return ALSGD_OK;
}

int alsgd_sched_destroy(alsgd_sched* s) {
    delete s;
    return ALSGD_OK;
}

int alsgd_sched_dispatch(alsgd_sched* s, uint32_t worker, double duration, uint32_t local_updates) {
    if (!s || !(duration > 0.0) || !std::isfinite(duration)) return ALSGD_E_ARG;
    if (worker >= s->n) return ALSGD_E_RANGE;
    Job& j = s->jobs[worker];
    if (j.in_flight) return ALSGD_E_STATE;
    const double start = j.ran_before ? j.restart_time : 0.0;
    j.completed_time = start + duration;
    j.local_updates = local_updates;
    j.in_flight = true;
    j.ran_before = true;
    return ALSGD_OK;
}

int alsgd_sched_next_batch(alsgd_sched* s, uint32_t* ids_out, double* times_out, uint32_t cap,
                           uint32_t* k_out, double* restart_out) {
    if (!s || !ids_out || !k_out) return ALSGD_E_ARG;
    *k_out = 0;
    if (s->t_max && s->t_local >= s->t_max) return ALSGD_OK;
    // Jobs in flight, earliest completion first, lower id first on equal times.
    std::vector<uint32_t> order;
    for (uint32_t w = 0; w < s->n; ++w)
        if (s->jobs[w].in_flight) order.push_back(w);
    if (order.empty()) return ALSGD_E_STATE;
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
        return s->jobs[a].completed_time < s->jobs[b].completed_time;
    });
    // The first one opens the grace window (tau_sync); later ones join while they finish inside it.
    const double tau_sync = s->jobs[order[0]].completed_time;
    uint32_t k = 0;
    uint64_t t_local = s->t_local;
    for (uint32_t w : order) {
        if (s->t_max && t_local >= s->t_max) break;
        if (k > 0 && !(s->jobs[w].completed_time - tau_sync <= s->tau_grace)) break;
        ++k;
        t_local += s->jobs[w].local_updates;
    }
    if (k > cap) return ALSGD_E_NOMEM;
    const double restart = tau_sync + s->tau_grace;
    for (uint32_t i = 0; i < k; ++i) {
        Job& j = s->jobs[order[i]];
        ids_out[i] = order[i];
        if (times_out) times_out[i] = j.completed_time;
        j.in_flight = false;
        j.restart_time = restart;
    }
    s->t_local = t_local;
    *k_out = k;
    if (restart_out) *restart_out = restart;
    return ALSGD_OK;
}

namespace {

// Image of a scheduler: header, then one record per worker.  Plain fixed-width fields, host byte order.
struct SchedImageHeader {
    char magic[8];
    uint32_t version;
    uint32_t n_workers;
    double tau_grace;
    uint64_t t_max;
    uint64_t t_local;
};
struct SchedImageJob {
    double completed_time;
    double restart_time;
    uint32_t local_updates;
    uint8_t in_flight;
    uint8_t ran_before;
    uint8_t reserved[2];
};
const char kSchedMagic[8] = {'A', 'L', 'S', 'G', 'D', 'S', 'C', '1'};

}  // namespace

int alsgd_sched_state_bytes(alsgd_sched* s, uint64_t* bytes_out) {
    if (!s || !bytes_out) return ALSGD_E_ARG;
    *bytes_out = sizeof(SchedImageHeader) + sizeof(SchedImageJob) * (uint64_t)s->n;
    return ALSGD_OK;
}

int alsgd_sched_export(alsgd_sched* s, void* host_dst, uint64_t bytes) {
    if (!s || !host_dst) return ALSGD_E_ARG;
    if (bytes < sizeof(SchedImageHeader) + sizeof(SchedImageJob) * (uint64_t)s->n) return ALSGD_E_NOMEM;
    SchedImageHeader h{};
    std::memcpy(h.magic, kSchedMagic, 8);
    h.version = 1; h.n_workers = s->n; h.tau_grace = s->tau_grace; h.t_max = s->t_max; h.t_local = s->t_local;
    uint8_t* out = static_cast<uint8_t*>(host_dst);
    std::memcpy(out, &h, sizeof(h));
    out += sizeof(h);
    for (const Job& j : s->jobs) {
        SchedImageJob r{};
        r.completed_time = j.completed_time; r.restart_time = j.restart_time; r.local_updates = j.local_updates;
        r.in_flight = j.in_flight ? 1 : 0; r.ran_before = j.ran_before ? 1 : 0;
        std::memcpy(out, &r, sizeof(r));
        out += sizeof(r);
    }
    return ALSGD_OK;
}

int alsgd_sched_import(alsgd_sched* s, const void* host_src, uint64_t bytes) {
    if (!s || !host_src || bytes < sizeof(SchedImageHeader)) return ALSGD_E_ARG;
    const uint8_t* in = static_cast<const uint8_t*>(host_src);
    SchedImageHeader h;
    std::memcpy(&h, in, sizeof(h));
    if (std::memcmp(h.magic, kSchedMagic, 8) != 0 || h.version != 1 || h.n_workers != s->n) return ALSGD_E_ARG;
    if (bytes < sizeof(SchedImageHeader) + sizeof(SchedImageJob) * (uint64_t)s->n) return ALSGD_E_ARG;
    if (!(h.tau_grace >= 0.0) || !std::isfinite(h.tau_grace)) return ALSGD_E_ARG;
    in += sizeof(h);
    std::vector<Job> jobs(s->n);
    for (uint32_t w = 0; w < s->n; ++w) {
        SchedImageJob r;
        std::memcpy(&r, in + sizeof(r) * (uint64_t)w, sizeof(r));
        if (r.in_flight > 1 || r.ran_before > 1 || !std::isfinite(r.completed_time) || !std::isfinite(r.restart_time)) return ALSGD_E_ARG;
        jobs[w].completed_time = r.completed_time; jobs[w].restart_time = r.restart_time;
        jobs[w].local_updates = r.local_updates; jobs[w].in_flight = r.in_flight != 0; jobs[w].ran_before = r.ran_before != 0;
    }
    s->jobs.swap(jobs);
    s->tau_grace = h.tau_grace; s->t_max = h.t_max; s->t_local = h.t_local;
    return ALSGD_OK;
}

int alsgd_sched_local_updates(alsgd_sched* s, uint64_t* t_local_out) {
    if (!s || !t_local_out) return ALSGD_E_ARG;
    *t_local_out = s->t_local;
    return ALSGD_OK;
}

}  // extern "C"

// CPU oracle for the asynchronous Local-SGD server step and the workers' inner AdamW step.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, single-threaded, scalar statement of what the
// CUDA library must compute.  It shares no code, header, table or constant with the CUDA path and
// is linked by nothing but the test-suite, the smoke check and the benchmark's CPU-baseline leg.
//
// Every floating-point expression below is written with one IEEE-754 binary32 operation per
// parenthesis pair, in the order the paper's Algorithm 3 states them; the file is compiled with
// -ffp-contract=off so that no multiply-add is fused.
//
// What pins each function (see tests/test_oracle_*.py):
//   orc_dn_arrive   hand traces of Algorithm 3, Eq. 4 (N = 1), Eq. 5 coefficients, beta = 0 -> plain
//                   SGD, buffer-sum invariant, one-cycle closed form, DiLoCo equivalence.
//   orc_adamw       hand case, sign-step property, pure-decay geometric sequence, undecayed tensors.
//                   The paper prints no AdamW formula; the variant is the textbook decoupled one.
//   orc_bf16_rne    exhaustive check against nearest-neighbour search over a strided 2^32 sweep.
//   orc_pg_norm2    hand values against the dispatch snapshot and against the running theta (decoy snapshot), the
//                   second arrival of a batch against theta after the first, NaN / Inf flagged.
//   orc_dylu        Eq. 6 values for speeds 1:1.5:2:3, H = 50.
//   orc_lr_at       Eq. 3 end points and clamps.
//   orc_schedule    Algorithm 2 + Algorithm 5 on hand timelines (Fig. 3 description).
//   orc_shard_probs Eq. 2 hand values, normalisation, start-up and balanced special cases.
//   orc_poly_weight, weight / dc_lambda / buffered arguments of orc_dn_arrive: formulas of Section 4
//                   ("Existing Fixes"): hand cases, zero-drift and homogeneity properties, buffered
//                   N = 1 == Eq. 4, buffered == Delayed Nesterov at cycle ends; SGD Momentum outer step:
//                   hand trace, theta' = theta - eps m', beta = 0 == plain SGD, geometric closed form.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

extern "C" {

// ---------------------------------------------------------------------------------------------
// bf16 round-to-nearest-even of a binary32 bit pattern (replica cast of the re-seed and of AdamW).
// NaN maps to a quiet NaN with the sign kept; overflow rounds to infinity.
// ---------------------------------------------------------------------------------------------
uint16_t orc_bf16_rne(uint32_t bits) {
    const uint32_t exponent = (bits >> 23) & 0xFFu;
    const uint32_t mantissa = bits & 0x7FFFFFu;
    if (exponent == 0xFFu && mantissa != 0u) {
        return (uint16_t)(((bits >> 16) & 0x8000u) | 0x7FC0u);
    }
    const uint32_t keep = bits >> 16;           // truncated value
    const uint32_t rest = bits & 0xFFFFu;       // discarded 16 bits
    uint32_t rounded = keep;
    if (rest > 0x8000u) {
        rounded = keep + 1u;                    // above the midpoint: up
    } else if (rest == 0x8000u) {
        if (keep & 1u) rounded = keep + 1u;     // tie: to the even mantissa
    }
    return (uint16_t)rounded;
}

static inline uint32_t f2u(float x) { uint32_t u; std::memcpy(&u, &x, 4); return u; }

void orc_cast_bf16(const float* src, uint16_t* dst, uint64_t lo, uint64_t hi) {
    for (uint64_t i = lo; i < hi; ++i) dst[i] = orc_bf16_rne(f2u(src[i]));
}

// ---------------------------------------------------------------------------------------------
// Scalars of Algorithm 3 derived from (N, beta, c): each is evaluated once in double and rounded
// to binary32 once.
// ---------------------------------------------------------------------------------------------
float orc_inv_n(uint32_t N) { return 1.0f / (float)N; }
float orc_boundary_weight(uint32_t N, float beta, float c) {     // (1 - cN + c) * beta
    return (float)((1.0 - (double)c * (double)N + (double)c) * (double)beta);
}
float orc_between_weight(float beta, float c) {                   // c * beta
    return (float)((double)c * (double)beta);
}

// ---------------------------------------------------------------------------------------------
// One arrival of Algorithm 3 ("Delayed Nesterov") for one worker, elements [lo, hi).
//   t           server updates applied so far (the algorithm's t before this arrival)
//   pg_current  0: pseudo-gradient against the parameters the worker was seeded with (base),
//                  Algorithm 1's delta = theta^(t-1) - theta_i;
//               1: against the running global parameters at this arrival.
//   weight      multiplies the pseudo-gradient first (1.0f: no staleness weighting; the multiply
//               is skipped entirely when weight == 1.0f).
//   dc_lambda   delay-compensation strength (Section 4, fix 3); 0 disables it.
//   buffered    1: "Async. Buffer" (Section 4, fix 4): theta moves only at the boundary, by one
//               Nesterov step (Eq. 4) on the buffer mean.
//               2: the same buffered structure with the "SGD Momentum" outer step of Section 4's
//               optimizer grid, which the text under Eq. 4 defines by its difference from Nesterov:
//               momentum weight beta instead of beta^2, gradient weight 1 instead of 1 + beta, i.e.
//               m' = beta m + g, theta' = theta - eps (beta m + g).  N = 1 applies it at every arrival.
// Returns 1 when this arrival is a momentum boundary ((t+1) % N == 0), else 0.
// ---------------------------------------------------------------------------------------------
int orc_dn_arrive(float* theta, float* m, float* Delta, const float* base, const float* p,
                  uint64_t lo, uint64_t hi, uint64_t t, uint32_t N, float beta, float eps, float c,
                  int pg_current, float weight, float dc_lambda, int buffered) {
    const int boundary = ((t + 1) % (uint64_t)N == 0) ? 1 : 0;
    const float invN = orc_inv_n(N);
    const float cb = orc_boundary_weight(N, beta, c);
    const float cn = orc_between_weight(beta, c);
    for (uint64_t i = lo; i < hi; ++i) {
        const float start = pg_current ? theta[i] : base[i];
        float g = start - p[i];                                   // pseudo-gradient
        if (dc_lambda != 0.0f) {                                  // g + lambda * g*g*(theta_now - theta_then)
            const float drift = theta[i] - start;
            g = g + ((dc_lambda * (g * g)) * drift);
        }
        if (weight != 1.0f) g = weight * g;
        const float d = Delta[i] + g;                             // Delta <- Delta + g_t
        const float gn = g * invN;                                // g_t / N
        if (buffered) {
            if (boundary) {
                const float mean = d * invN;
                const float mn = (beta * m[i]) + mean;            // Eq. 4, momentum
                float u;
                if (buffered == 2) {
                    u = (beta * m[i]) + mean;                     // SGD Momentum: weights beta and 1
                } else {
                    u = ((beta * beta) * m[i]) + ((1.0f + beta) * mean);   // Nesterov: beta^2 and 1 + beta
                }
                theta[i] = theta[i] - (eps * u);
                m[i] = mn;
                Delta[i] = 0.0f;
            } else {
                Delta[i] = d;
            }
            continue;
        }
        if (boundary) {
            const float mn = (beta * m[i]) + (d * invN);          // m_{t+1} = beta m_t + Delta/N
            const float u = (cb * mn) + gn;                       // (1-cN+c) beta m_{t+1} + g_t/N
            theta[i] = theta[i] - (eps * u);
            m[i] = mn;
            Delta[i] = 0.0f;
        } else {
            const float u = (c == 0.0f) ? gn : ((cn * m[i]) + gn); // c beta m_t + g_t/N
            theta[i] = theta[i] - (eps * u);
            Delta[i] = d;
        }
    }
    return boundary;
}

// Optional diagnostics of one arrival: sum of squared pseudo-gradient entries (double) and whether
// any entry is not finite.  Not in the paper; a by-product the library can report.
double orc_pg_norm2(const float* theta, const float* base, const float* p, uint64_t lo, uint64_t hi,
                    int pg_current, uint32_t* nonfinite) {
    double acc = 0.0;
    uint32_t bad = 0;
    for (uint64_t i = lo; i < hi; ++i) {
        const float start = pg_current ? theta[i] : base[i];
        const float g = start - p[i];
        if (!std::isfinite(g)) bad = 1;
        acc += (double)g * (double)g;
    }
    if (nonfinite) *nonfinite = bad;
    return acc;
}

// Re-seed at dispatch (Algorithm 2's train(W_completed, theta); Algorithm 1's theta_i <- theta):
// the worker's parameters, its dispatch snapshot and its bf16 replica all become the global model.
// Either output pointer may be null.
void orc_reseed(const float* theta, float* p, float* base, uint16_t* replica, uint64_t lo, uint64_t hi) {
    for (uint64_t i = lo; i < hi; ++i) {
        if (p) p[i] = theta[i];
        if (base) base[i] = theta[i];
        if (replica) replica[i] = orc_bf16_rne(f2u(theta[i]));
    }
}

// ---------------------------------------------------------------------------------------------
// One AdamW step (decoupled weight decay, bias-corrected, epsilon outside the root) on elements
// [lo, hi) of one worker.  decay[i] != 0 marks weight-decayed elements.  step >= 1 is the worker's
// lifetime step count (the optimizer state is never reset between rounds).
// ---------------------------------------------------------------------------------------------
void orc_adamw(float* p, float* m, float* v, const float* g, uint16_t* replica, const uint8_t* decay,
               uint64_t lo, uint64_t hi, uint64_t step, float lr, float b1, float b2, float eps, float wd) {
    const float bc1 = (float)(1.0 - std::pow((double)b1, (double)step));
    const float bc2 = (float)(1.0 - std::pow((double)b2, (double)step));
    const float omb1 = 1.0f - b1;
    const float omb2 = 1.0f - b2;
    for (uint64_t i = lo; i < hi; ++i) {
        const float gi = g[i];
        const float mi = (b1 * m[i]) + (omb1 * gi);
        const float vi = (b2 * v[i]) + (omb2 * (gi * gi));
        m[i] = mi;
        v[i] = vi;
        const float mh = mi / bc1;
        const float vh = vi / bc2;
        const float r = mh / (std::sqrt(vh) + eps);
        float pi = p[i];
        if (decay && decay[i]) {
            pi = pi - (lr * (r + (wd * pi)));
        } else {
            pi = pi - (lr * r);
        }
        p[i] = pi;
        if (replica) replica[i] = orc_bf16_rne(f2u(pi));
    }
}

// ---------------------------------------------------------------------------------------------
// Eq. 6, Dynamic Local Updates: steps_w = floor(v_w / max v * H), never below one step.
// ---------------------------------------------------------------------------------------------
void orc_dylu(const double* speeds, uint32_t n, uint32_t H, uint32_t* steps) {
    double vmax = 0.0;
    for (uint32_t w = 0; w < n; ++w) if (speeds[w] > vmax) vmax = speeds[w];
    for (uint32_t w = 0; w < n; ++w) {
        const double x = std::floor((speeds[w] / vmax) * (double)H);
        steps[w] = x < 1.0 ? 1u : (uint32_t)x;
    }
}

// ---------------------------------------------------------------------------------------------
// Eq. 3: linear warm-up then cosine decay to eta_min; the cosine's argument ratio is clamped to
// [0, 1] and T - t_warmup to >= 0 (a zero-length decay counts as finished).
// ---------------------------------------------------------------------------------------------
double orc_lr_at(double eta_max, double eta_min, uint64_t t_warmup, uint64_t T, uint64_t t) {
    if (t < t_warmup) return (double)t * eta_max / (double)t_warmup;
    const double span = T > t_warmup ? (double)(T - t_warmup) : 0.0;
    double ratio = span > 0.0 ? (double)(t - t_warmup) / span : 1.0;
    if (ratio < 0.0) ratio = 0.0;
    if (ratio > 1.0) ratio = 1.0;
    const double pi = 3.14159265358979323846;
    return eta_min + 0.5 * (eta_max - eta_min) * (1.0 + std::cos(ratio * pi));
}

// ---------------------------------------------------------------------------------------------
// Eq. 2, data-shard sampling: p_i proportional to max(|D_i| / sum|D_j| - n_i / sum n_j, 0), with n_i the
// number of data points already learned from shard i.  Before anything was learned (sum n = 0) the
// learned share counts as zero; if no shard is under-sampled (all terms zero) the size shares are used.
// ---------------------------------------------------------------------------------------------
void orc_shard_probs(const double* sizes, const double* learned, uint32_t n, double* probs) {
    double total_size = 0.0, total_learned = 0.0;
    for (uint32_t i = 0; i < n; ++i) { total_size += sizes[i]; total_learned += learned[i]; }
    double norm = 0.0;
    for (uint32_t i = 0; i < n; ++i) {
        const double size_share = sizes[i] / total_size;
        const double learned_share = total_learned > 0.0 ? learned[i] / total_learned : 0.0;
        const double gap = size_share - learned_share;
        probs[i] = gap > 0.0 ? gap : 0.0;
        norm += probs[i];
    }
    for (uint32_t i = 0; i < n; ++i) probs[i] = norm > 0.0 ? probs[i] / norm : sizes[i] / total_size;
}

// Staleness weight of "Async. DiLoCo + Poly": (1 + staleness)^(-0.5), rounded to binary32.
float orc_poly_weight(uint64_t staleness) {
    return (float)std::pow(1.0 + (double)staleness, -0.5);
}

// ---------------------------------------------------------------------------------------------
// Algorithm 2 (task scheduling) with Algorithm 5 (get_worker) on faked time.
//   durations[w * n_rounds + r]  training time of worker w's r-th job
//   local_updates[w]             inner steps per job of worker w (added to t_local at sync)
// All workers start at time 0.  The loop runs while t_local < t_max and fewer than max_arrivals
// arrivals were produced.  Outputs per arrival: worker id, completion time, index of its batch
// (one batch = one grace window = the list W_completed between two re-dispatches).
// Returns the number of arrivals written.
// ---------------------------------------------------------------------------------------------
uint32_t orc_schedule(uint32_t n_workers, const double* durations, uint32_t n_rounds,
                      const uint32_t* local_updates, double tau_grace, uint64_t t_max,
                      uint32_t max_arrivals, uint32_t* out_worker, double* out_time, uint32_t* out_batch) {
    const double INF = std::numeric_limits<double>::infinity();
    std::vector<double> completed_time(n_workers);
    std::vector<uint32_t> round(n_workers, 0);
    std::vector<char> pending(n_workers, 1);          // job running or finished, not yet synced
    std::vector<uint32_t> W_completed;
    for (uint32_t w = 0; w < n_workers; ++w) completed_time[w] = 0.0 + durations[(uint64_t)w * n_rounds + 0];
    uint64_t t_local = 0;
    double tau_sync = INF;
    uint32_t n_out = 0, batch = 0;
    while (t_local < t_max && n_out < max_arrivals) {
        // get_worker(): earliest completed worker not yet processed, if inside the grace period
        int64_t w = -1;
        for (uint32_t u = 0; u < n_workers; ++u) {
            if (!pending[u]) continue;
            if (w < 0 || completed_time[u] < completed_time[w]) w = u;   // ties: lower id stays
        }
        if (w >= 0 && !(tau_sync == INF || completed_time[w] - tau_sync <= tau_grace)) w = -1;
        if (w >= 0) {
            if (completed_time[w] < tau_sync) tau_sync = completed_time[w];
            out_worker[n_out] = (uint32_t)w;          // theta <- sync(theta, w.update)
            out_time[n_out] = completed_time[w];
            out_batch[n_out] = batch;
            ++n_out;
            pending[w] = 0;
            W_completed.push_back((uint32_t)w);
            t_local += local_updates[w];
        } else {
            const double restart = tau_sync + tau_grace;
            tau_sync = INF;
            for (uint32_t u : W_completed) {          // train(W_completed, theta)
                round[u] += 1;
                if (round[u] >= n_rounds) return n_out;   // ran out of supplied durations
                completed_time[u] = restart + durations[(uint64_t)u * n_rounds + round[u]];
                pending[u] = 1;
            }
            W_completed.clear();
            ++batch;
        }
    }
    return n_out;
}

}  // extern "C"

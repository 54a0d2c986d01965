/*
 * alsgd.h — C ABI of the asynchronous Local-SGD server step and the workers' inner AdamW step,
 * on one NVIDIA B200 (sm_100a).
 *
 * The library keeps, in one caller-owned device arena, the server state of the paper's Algorithm 3
 * ("Delayed Nesterov": global parameters theta, momentum m, buffer Delta, update counter t) and W
 * simulated workers (fp32 parameters, the fp32 snapshot they were dispatched with, AdamW moments,
 * a bf16 replica), all as flat vectors of P elements laid out from a tensor table.
 *
 * Conventions
 *   - Every function returns ALSGD_OK (0) or a negative alsgd_status.  Nothing throws, aborts,
 *     traps or prints.  Arguments are checked before anything is enqueued, so ALSGD_E_ARG, _RANGE,
 *     _STATE, _NOMEM and _UNSUPPORTED leave the context exactly as it was.  ALSGD_E_CUDA from a call
 *     whose first launch failed does too; if a later launch of the same call fails (an arrival batch
 *     larger than one pass, a host gradient copied in pieces) the device state is already ahead of
 *     the host bookkeeping: the context then refuses every further state-changing call with
 *     ALSGD_E_STATE and can only be read, destroyed or re-filled by alsgd_import_state.
 *   - "host" / "device" is stated for every pointer.  The arena and the stream belong to the
 *     caller; the context owns only host bookkeeping.  No entry point allocates device memory
 *     (alsgd_init and alsgd_destroy allocate and free host memory only).
 *   - Calls enqueue work on the context's stream and return without waiting, except where a
 *     host output needs the result (stated per call).  A context is not thread-safe.
 *   - All element counts and indices are 64-bit.
 */
#ifndef ALSGD_H
#define ALSGD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum alsgd_status {
    ALSGD_OK = 0,
    ALSGD_E_ARG = -1,    /* invalid argument (null pointer, zero size, value outside its domain) */
    ALSGD_E_RANGE = -2,  /* worker id or index out of range */
    ALSGD_E_STATE = -3,  /* call not allowed in the current state (e.g. arrival of a worker never dispatched) */
    ALSGD_E_CUDA = -4,   /* a CUDA runtime call failed; see alsgd_last_cuda_error */
    ALSGD_E_NOMEM = -5,  /* arena too small, or host allocation failed */
    ALSGD_E_UNSUPPORTED = -6,
    ALSGD_E_BOUNDS = -7  /* debug build only: a kernel access fell outside the arena and was skipped (alsgd_sync) */
} alsgd_status;

/* Text for a status code (static storage, host). */
const char* alsgd_strerror(int status);

/* ------------------------------------------------------------------------------------------------
 * Flat-buffer layout.  The paper treats the model as one parameter vector theta (Algorithm 3 acts
 * on it elementwise); the tensor table only says where each tensor lives in that vector and whether
 * the inner optimizer applies weight decay to it (Table 5: weight decay 0.1).
 * ---------------------------------------------------------------------------------------------- */
#define ALSGD_TENSOR_DECAY 1u

typedef struct alsgd_tensor_desc {
    uint64_t numel;   /* > 0 */
    uint32_t flags;   /* ALSGD_TENSOR_DECAY or 0 */
    uint32_t reserved;
} alsgd_tensor_desc;

/* Offsets of n tensors in the flat vector: tensor i starts at the next multiple of align_elems
 * (>= 1) after tensor i-1; *P_out is the padded total (a multiple of align_elems).  Padding
 * elements are zero, are never weight-decayed and take part in nothing observable.
 * tensors: host, n entries.  offsets_out: host, n entries, may be NULL.  ALSGD_E_ARG on n = 0,
 * numel = 0, align_elems = 0 or 64-bit overflow. */
int alsgd_layout_size(const alsgd_tensor_desc* tensors, uint32_t n, uint32_t align_elems,
                      uint64_t* P_out, uint64_t* offsets_out);

/* ------------------------------------------------------------------------------------------------
 * Context
 * ---------------------------------------------------------------------------------------------- */
typedef struct alsgd_ctx alsgd_ctx;

/* Which model the pseudo-gradient of an arriving worker is taken against. */
#define ALSGD_PG_DISPATCH 0u  /* the model the worker was seeded with: delta = theta^(t-1) - theta_i (Algorithm 1) */
#define ALSGD_PG_CURRENT 1u   /* the running global model at the moment of that arrival */

#define ALSGD_CFG_REPLICA_BF16 1u  /* keep a bf16 copy of every worker's parameters */
#define ALSGD_CFG_GRAD_STAGING 2u  /* reserve a P-element fp32 staging buffer so that alsgd_inner_adamw accepts host gradients */
#define ALSGD_CFG_OUTER_BUFFERED 4u /* "Async. Buffer" of Section 4 instead of Delayed Nesterov: Delta accumulates every arrival,
                                       theta and m move only on every N-th, by the Nesterov step of Eq. 4 on Delta/N; c is unused */
#define ALSGD_CFG_OUTER_SGDM 8u     /* "SGD Momentum" of Section 4's outer-optimizer grid, in the same buffered structure: on every
                                       N-th arrival m <- beta m + g, theta <- theta - eps (beta m + g) with g = Delta/N, i.e. Eq. 4
                                       with beta in place of beta^2 and 1 in place of 1 + beta (the text under Eq. 4).  N = 1 applies
                                       it at every arrival, as the paper's grid did; beta = 0 is plain outer SGD.  c is unused.
                                       Not together with ALSGD_CFG_OUTER_BUFFERED. */
#define ALSGD_CFG_STABLE_PTRS 16u   /* no deferred stores: every worker keeps a snapshot of its own and its parameters are written
                                       at every dispatch, Delta's zeros are written at every boundary, so the pointers of
                                       alsgd_state_ptrs / alsgd_worker_state_ptrs stay valid and current for the context's lifetime.
                                       Costs 4 (parameters) + 4 (own snapshot) bytes per parameter per dispatched worker instead of
                                       4 per window, and 4 per boundary. */

typedef struct alsgd_config {
    uint32_t n_workers;  /* W >= 1 replicas resident in the arena */
    uint32_t N;          /* Algorithm 3 buffer size (the "delay period" of Table 5), >= 1 */
    uint32_t pg_base;    /* ALSGD_PG_DISPATCH or ALSGD_PG_CURRENT */
    uint32_t flags;      /* ALSGD_CFG_* */
    float beta;          /* momentum decay, [0, 1) */
    float outer_lr;      /* epsilon of Algorithm 3 */
    float c;             /* momentum activation, [0, 1/N] (Algorithm 3; default 0) */
    float adam_b1, adam_b2, adam_eps, adam_wd; /* inner AdamW: betas in [0,1), eps >= 0, wd >= 0 */
    int32_t device;      /* CUDA device ordinal that owns arena and stream */
    void* stream;        /* cudaStream_t (0 = legacy default stream); caller-owned */
    void* arena;         /* device, 256-byte aligned, caller-owned for the context's lifetime */
    uint64_t arena_bytes;
} alsgd_config;

/* Bytes of arena needed for a layout and configuration (pure host arithmetic). */
int alsgd_arena_bytes(const alsgd_tensor_desc* tensors, uint32_t n, uint32_t align_elems,
                      const alsgd_config* cfg, uint64_t* bytes_out);

/* Create a context in the state Algorithm 3 starts from: t = 0, m = 0, Delta = 0; theta = 0 until
 * alsgd_set_global; every worker is "never dispatched" with zero AdamW moments.  Enqueues the zero
 * fills on cfg->stream.  ALSGD_E_ARG for values outside the domains above or a misaligned arena,
 * ALSGD_E_NOMEM if arena_bytes is too small. */
int alsgd_init(alsgd_ctx** out, const alsgd_tensor_desc* tensors, uint32_t n, uint32_t align_elems,
               const alsgd_config* cfg);

/* Free the host bookkeeping (and, with ALSGD_CFG_GRAD_STAGING, the context's internal copy stream, after
 * waiting for it).  Never touches the arena.  Does not wait for the caller's stream: kernels of earlier
 * calls may still be running on it, so the caller synchronises that stream (or calls alsgd_sync first)
 * before it frees or reuses the arena. */
int alsgd_destroy(alsgd_ctx* ctx);

/* Load theta^(0) (Algorithm 2: theta <- theta^(0)) / read theta.  P floats; is_device says where the
 * caller's buffer lives.  Host buffers: the copy is enqueued and the call waits for it. */
int alsgd_set_global(alsgd_ctx* ctx, const float* src, int src_is_device);
int alsgd_get_global(alsgd_ctx* ctx, float* dst, int dst_is_device);

/* Overwrite / read one worker's fp32 parameters (a test and simulation hook: it stands in for the
 * forward/backward passes this library does not run).  Same pointer rules as alsgd_set_global. */
int alsgd_set_worker_params(alsgd_ctx* ctx, uint32_t worker, const float* src, int src_is_device);
int alsgd_get_worker_params(alsgd_ctx* ctx, uint32_t worker, float* dst, int dst_is_device);

/* Dispatch one worker with the current server model (Algorithm 2, train(W, theta); Algorithm 1,
 * theta_i <- theta): its parameters, its dispatch snapshot and its bf16 replica become theta; its
 * pull tick becomes t.  AdamW moments and step count are untouched (the paper keeps the inner
 * optimizer state on the worker across rounds and never resets it).  ALSGD_E_RANGE for a bad id. */
int alsgd_pull(alsgd_ctx* ctx, uint32_t worker);

/* One inner AdamW step of one worker (InnerOpt of Algorithm 1; decoupled weight decay on tensors
 * flagged ALSGD_TENSOR_DECAY, bias correction from `step`, epsilon outside the root), followed by
 * the bf16 cast of the new parameters into the replica.
 *   grads            P fp32 values, 16-byte aligned, device or host (host needs
 *                    ALSGD_CFG_GRAD_STAGING; the vector is copied in pieces on an internal stream and the
 *                    step on each piece is enqueued on the context's stream behind its copy, so copy and
 *                    arithmetic overlap; the buffer is borrowed until the context's stream has passed
 *                    this call; pinned memory keeps the call asynchronous)
 *   step             the worker's lifetime step count, >= 1
 *   lr               learning rate of this step
 * ALSGD_E_STATE if the worker was never dispatched, ALSGD_E_ARG if step = 0. */
int alsgd_inner_adamw(alsgd_ctx* ctx, uint32_t worker, const float* grads, int grads_is_device,
                      uint64_t step, float lr);

/* The same step with gradients stored as bf16 bit patterns (widened exactly to fp32 before use), as a
 * mixed-precision backward pass produces them: 28 instead of 30 bytes per parameter on the device and half the
 * host-to-device traffic.  The paper states no gradient precision; this is an option beside the fp32 call. */
int alsgd_inner_adamw_bf16(alsgd_ctx* ctx, uint32_t worker, const uint16_t* grads, int grads_is_device,
                           uint64_t step, float lr);

#define ALSGD_ARRIVE_RESEED 1u    /* re-dispatch all k workers with the final theta (Algorithm 2, the branch taken when get_worker() finds nobody) */
#define ALSGD_ARRIVE_NORM 2u      /* report the squared norm of each pseudo-gradient */
#define ALSGD_ARRIVE_NANCHECK 4u  /* report whether each pseudo-gradient has a non-finite entry */

typedef struct alsgd_arrival_info {
    uint64_t tick;       /* Algorithm 3's t at which this arrival was applied */
    uint64_t staleness;  /* tick minus the worker's pull tick */
    double gnorm2;       /* sum of squared pseudo-gradient entries (0 unless NORM); squares are formed in binary32, so an
                            entry beyond 1.8e19 in magnitude makes it +inf although the entry is finite */
    uint32_t worker;
    uint32_t boundary;   /* 1 if (t+1) % N == 0: momentum updated, buffer reset */
    uint32_t nonfinite;  /* 1 if any entry was NaN or Inf (0 unless NANCHECK) */
    uint32_t dropped;    /* 1 if the update was discarded as too stale (alsgd_arrive_ex, ALSGD_STALE_POLY_THRES) */
} alsgd_arrival_info;

/* The sync() of Algorithm 2 for the k workers of one grace window, in the given order: for each,
 * pseudo-gradient -> Delta += g -> on every N-th server update m <- beta m + Delta/N,
 * theta <- theta - eps((1-cN+c) beta m + g/N), Delta <- 0; otherwise theta <- theta - eps(c beta m + g/N)
 * (Algorithm 3); t advances by k.  The k arrivals are applied in one pass over memory and give
 * exactly the result of k single calls.  With RESEED all k workers are then dispatched again with
 * the final theta.
 *   worker_ids   host, k entries, copied at call time
 *   info         host, k entries or NULL.  With NORM or NANCHECK and info != NULL the call waits for
 *                the stream; otherwise it only enqueues.
 * k = 0 is a no-op.  ALSGD_E_ARG: k > W, a duplicate id.  ALSGD_E_RANGE: id >= W.  ALSGD_E_STATE: a
 * worker that is not currently dispatched (never pulled, or already arrived and not re-dispatched). */
int alsgd_arrive(alsgd_ctx* ctx, const uint32_t* worker_ids, uint32_t k, uint32_t flags,
                 alsgd_arrival_info* info);

/* Staleness handling of Section 4 ("Existing Fixes"), staleness = server updates since the worker's dispatch. */
#define ALSGD_STALE_NONE 0u
#define ALSGD_STALE_POLY 1u        /* g <- (1 + staleness)^-0.5 * g  ("Async. DiLoCo + Poly") */
#define ALSGD_STALE_POLY_THRES 2u  /* Poly, and updates with staleness > stale_threshold are discarded ("PolyThres") */

typedef struct alsgd_arrive_opts {
    const float* weights;      /* host, k entries or NULL: g_j <- weights[j] * g_j (ignored when a staleness rule is set) */
    float dc_lambda;           /* delay compensation (Section 4): g <- g + lambda * g*g*(theta_now - theta_at_dispatch); 0 = off */
    uint32_t staleness_rule;   /* ALSGD_STALE_* */
    uint32_t stale_threshold;  /* for ALSGD_STALE_POLY_THRES (the paper uses 10) */
    uint32_t reserved;
} alsgd_arrive_opts;

/* alsgd_arrive with the pseudo-gradient modifications of Section 4.  The pseudo-gradient of each arrival is
 * first delay-compensated, then weighted, then enters Algorithm 3 (or the buffered outer step) unchanged
 * otherwise; NORM / NANCHECK report the unmodified pseudo-gradient.  A discarded update (PolyThres) is not a
 * server update: t does not advance, info[j].dropped = 1, and with RESEED its worker is still re-dispatched.
 * opts == NULL behaves exactly like alsgd_arrive.  ALSGD_E_ARG: negative or non-finite dc_lambda, unknown
 * staleness rule, non-finite weight. */
int alsgd_arrive_ex(alsgd_ctx* ctx, const uint32_t* worker_ids, uint32_t k, uint32_t flags,
                    const alsgd_arrive_opts* opts, alsgd_arrival_info* info);

/* Server update counter t of Algorithm 3 and its phase t % N.  Either pointer may be NULL. */
int alsgd_counters(alsgd_ctx* ctx, uint64_t* t_out, uint32_t* phase_out);

typedef struct alsgd_ptrs {
    float* theta;  /* device, P */
    float* m;      /* device, P */
    float* delta;  /* device, P */
    uint64_t P;
    uint32_t n_workers;
    uint32_t reserved;
} alsgd_ptrs;

typedef struct alsgd_worker_ptrs {
    float* p;          /* device, P: the worker's parameters */
    float* base;       /* device, P: dispatch snapshot, read-only for the caller: workers dispatched in the same
                          window share one (NULL in ALSGD_PG_CURRENT mode) */
    float* adam_m;     /* device, P */
    float* adam_v;     /* device, P */
    uint16_t* replica; /* device, P bf16 bit patterns (NULL without ALSGD_CFG_REPLICA_BF16) */
} alsgd_worker_ptrs;

/* Borrowed device pointers into the arena, for a harness that perturbs workers and reads results.
 * theta, m, adam_m, adam_v and replica always hold the current state and stay valid until
 * alsgd_destroy.  `delta`, `p` and `base` are different: the library defers two stores and shares
 * snapshots, and makes the state good only at the moment of this call.
 *   - Right after a momentum boundary Delta is zero by definition but the zeros may not have been
 *     written; alsgd_state_ptrs enqueues the fill.  `delta` read after a LATER boundary without a new
 *     alsgd_state_ptrs call may show the pre-boundary buffer.
 *   - Right after a dispatch (alsgd_pull, alsgd_arrive with RESEED) a worker's parameters equal its
 *     snapshot and are not copied into `p`; alsgd_worker_state_ptrs enqueues that copy (P floats).
 *     A `p` pointer kept across a LATER dispatch of that worker shows the previous round's
 *     parameters until the next alsgd_worker_state_ptrs, alsgd_set_worker_params or AdamW step.
 *   - Workers dispatched in one window share one snapshot slot, and a slot is recycled when its last
 *     worker has been dispatched anew, so `base` is valid only until the next dispatch of ANY worker.
 * So: call the accessor again after every alsgd_pull / alsgd_arrive before touching delta, p or base;
 * writes through `p` are picked up by the next arrival or AdamW step of that worker.  A caller that
 * must hold the pointers creates the context with ALSGD_CFG_STABLE_PTRS, which makes all of them
 * permanent at the cost stated there. */
int alsgd_state_ptrs(alsgd_ctx* ctx, alsgd_ptrs* out);
int alsgd_worker_state_ptrs(alsgd_ctx* ctx, uint32_t worker, alsgd_worker_ptrs* out);

/* Checkpoint / resume.  The paper starts its runs from a pretrained checkpoint (Section 4; Table 5) and
 * keeps each worker's optimizer state across rounds, without describing a mechanism; this is the
 * library's.  The image holds the layout size, W, N, the pseudo-gradient mode, t, every worker's dispatch
 * state and pull tick, then theta, m, Delta and each worker's parameters, snapshot, AdamW moments and replica.
 *   alsgd_state_bytes     size of the image for this context
 *   alsgd_export_state    host_dst: host, `bytes` >= that size; waits for the stream
 *   alsgd_import_state    host_src: host image written by a context with the same layout size, W, N, mode
 *                         and replica setting (hyper-parameters may differ); replaces the whole state; waits
 * ALSGD_E_NOMEM: buffer too small.  ALSGD_E_ARG: not an image, or made for a different shape. */
int alsgd_state_bytes(alsgd_ctx* ctx, uint64_t* bytes_out);
int alsgd_export_state(alsgd_ctx* ctx, void* host_dst, uint64_t bytes);
int alsgd_import_state(alsgd_ctx* ctx, const void* host_src, uint64_t bytes);

/* Wait for the context's stream.  In the debug build of the library (libalsgd_dbg.so, compiled with
 * -DALSGD_DEBUG_BOUNDS: every kernel access to an arena-owned vector is checked against the arena's byte range
 * and its alignment, an offending access is skipped and recorded instead of faulting) it then reads the
 * record and returns ALSGD_E_BOUNDS if any access was refused since alsgd_init; the record is sticky. */
int alsgd_sync(alsgd_ctx* ctx);

/* Debug build: device address of the record alsgd_sync reads (one uint32, a bit per kind of vector: theta 1,
 * Delta 2, m 4, worker parameters 8, snapshots 16, re-seed targets 32, AdamW p/m/v 64/128/256, replica 512), so
 * that a caller can read or clear it.  Normal build: ALSGD_E_UNSUPPORTED and *word_out = NULL. */
int alsgd_debug_word_ptr(alsgd_ctx* ctx, uint32_t** word_out);

/* Debug build: from now on treat only the first `bytes` of the arena as in range (0 = the whole arena again), so
 * that the checks can be seen working without any access leaving the arena: accesses to the slices behind the
 * limit are refused and recorded although the memory is the caller's own.  ALSGD_E_ARG if bytes exceeds the
 * arena.  Normal build: ALSGD_E_UNSUPPORTED. */
int alsgd_debug_guard_limit(alsgd_ctx* ctx, uint64_t bytes);

/* cudaError_t of the most recent failed CUDA call of this context (0 if none). */
int alsgd_last_cuda_error(alsgd_ctx* ctx);

/* ------------------------------------------------------------------------------------------------
 * Host-side helpers of the method (no device work)
 * ---------------------------------------------------------------------------------------------- */

/* Dynamic Local Updates, Eq. 6: steps_w = floor(v_w / max v * H), at least 1.
 * speeds: host, n positive values (steps per second).  steps_out: host, n entries. */
int alsgd_dylu_steps(const double* speeds, uint32_t n, uint32_t H, uint32_t* steps_out);

/* Data-shard sampling, Eq. 2: probs_i proportional to max(sizes_i / sum sizes - learned_i / sum learned, 0),
 * learned_i = data points already learned from shard i, so that under-sampled shards are preferred.  While
 * nothing has been learned the learned share counts as 0; if no shard is under-sampled the size shares are
 * returned.  sizes (> 0), learned (>= 0), probs_out: host, n entries.  The draw itself is the caller's. */
int alsgd_shard_probs(const double* sizes, const double* learned, uint32_t n, double* probs_out);

typedef struct alsgd_lr_sched {
    double eta_max, eta_min;
    uint64_t t_warmup, T;
} alsgd_lr_sched;

/* Learning rate of Eq. 3 at shard-local step t: linear warm-up, then cosine decay to eta_min with
 * the ratio (t - t_warmup)/(T - t_warmup) kept inside [0, 1] and T - t_warmup >= 0. */
int alsgd_lr_at(const alsgd_lr_sched* sched, uint64_t t, double* lr_out);

/* Asynchronous task scheduling (Algorithm 2 with get_worker() of Algorithm 5) on faked time.
 * The caller plays train(): it dispatches a job for a worker with the time that job will take;
 * alsgd_sched_next_batch returns the workers the server synchronises in one grace window, in order. */
typedef struct alsgd_sched alsgd_sched;

/* tau_grace >= 0.  t_max: total local updates after which no further arrival is produced (0 = no limit). */
int alsgd_sched_create(alsgd_sched** out, uint32_t n_workers, double tau_grace, uint64_t t_max);
int alsgd_sched_destroy(alsgd_sched* s);

/* Start a job on an idle worker.  It starts at time 0 if the worker has never run, else at the moment
 * the grace window that synchronised it closed (tau_sync + tau_grace), and completes `duration`
 * (> 0) later; `local_updates` is added to t_local when it is synchronised.
 * ALSGD_E_STATE if the worker already has a job in flight. */
int alsgd_sched_dispatch(alsgd_sched* s, uint32_t worker, double duration, uint32_t local_updates);

/* Run Algorithm 2's loop until get_worker() returns null: collect the earliest completed worker (ties:
 * lower id) while its completion time is within tau_grace of the window's first, then close the window.
 *   ids_out, times_out   host, cap entries (times_out may be NULL)
 *   k_out                number of workers in the window (0 once t_local >= t_max)
 *   restart_out          time at which the returned workers start their next job (may be NULL)
 * The returned workers are idle until dispatched again.  ALSGD_E_STATE if no job is in flight,
 * ALSGD_E_NOMEM if cap is smaller than the window (nothing is consumed). */
int alsgd_sched_next_batch(alsgd_sched* s, uint32_t* ids_out, double* times_out, uint32_t cap,
                           uint32_t* k_out, double* restart_out);

/* Total local updates synchronised so far (Algorithm 2's t_local). */
int alsgd_sched_local_updates(alsgd_sched* s, uint64_t* t_local_out);

/* Checkpoint / resume of the scheduler, the counterpart of alsgd_export_state for Algorithm 2's own state:
 * tau_grace, t_max, t_local and per worker the job in flight (completion time, local updates), whether it ever
 * ran and the restart time its last window gave it (tau_sync + tau_grace).  An image imported into a scheduler
 * created for the same number of workers continues the timeline exactly where it stopped: the same windows, ids,
 * times and restart times.  All host memory; a few dozen bytes per worker.
 *   alsgd_sched_state_bytes   size of the image
 *   alsgd_sched_export        host_dst: `bytes` >= that size (ALSGD_E_NOMEM otherwise)
 *   alsgd_sched_import        ALSGD_E_ARG: not a scheduler image, another worker count, or fields outside their
 *                             domain; the scheduler is unchanged then */
int alsgd_sched_state_bytes(alsgd_sched* s, uint64_t* bytes_out);
int alsgd_sched_export(alsgd_sched* s, void* host_dst, uint64_t bytes);
int alsgd_sched_import(alsgd_sched* s, const void* host_src, uint64_t bytes);

/* ------------------------------------------------------------------------------------------------
 * Diagnostics without any allocation (the paper has no counterpart; this serves embedders)
 * ---------------------------------------------------------------------------------------------- */

/* Largest vector alsgd_pg_norm_static accepts. */
#define ALSGD_STATIC_MAX_ELEMS (1ull << 27)

/* Squared norm and non-finite flag of a pseudo-gradient start - p, for callers that cannot obtain
 * device memory of their own: code hosted inside another framework's memory plan or between its
 * graph launches, or a process whose device memory was all handed out at start-up.  It needs no
 * context and no arena.  Its working memory (one flag word plus one double per 4096 elements,
 * 256 KiB + 256 bytes in total) is a fixed array inside the library image, which every GPU that
 * loads the library holds until the process exits; the call itself invokes no allocating routine.
 *   start, p        device, n fp32 values each, 16-byte aligned, caller-owned (for a worker of a
 *                   context: its dispatch snapshot and its parameters)
 *   n               1 .. ALSGD_STATIC_MAX_ELEMS; more returns ALSGD_E_NOMEM and does nothing
 *   device, stream  the device that owns the buffers and the stream to enqueue on
 *   gnorm2_out      device, one double: sum of (start[i] - p[i])^2, accumulated in double in a fixed
 *                   order (the same inputs give the same bits on every call)
 *   nonfinite_out   device, one uint32: 1 if any entry of start - p is NaN or Inf, else 0
 * The call only enqueues; the outputs are valid once the stream reaches them.  The first call on each
 * device looks up the array's device address; make that first call outside any stream capture.  With the
 * CUDA runtime's default lazy module loading that first call is also the moment the device sets the array and
 * this entry point's kernels aside, so a process that hands out all of its device memory should make one
 * warm-up call (n = 4 on any two valid buffers is enough) at start-up, before it does so: afterwards no call
 * needs anything more.  The looked-up address is cached per device ordinal for the life of the process and
 * does not survive a reset of that device's primary context (cudaDeviceReset).
 * All calls on one device share the one array and it keeps the previous call's contents, so the call
 * clears what it accumulates into before use; two calls whose kernels can overlap on the GPU (other
 * streams, other threads) race on it and must be ordered by the caller.
 * ALSGD_E_ARG: null or misaligned pointer, n = 0.  ALSGD_E_RANGE: device ordinal outside 0..63. */
int alsgd_pg_norm_static(const float* start, const float* p, uint64_t n, int32_t device, void* stream,
                         double* gnorm2_out, uint32_t* nonfinite_out);

#ifdef __cplusplus
}
#endif
#endif /* ALSGD_H */

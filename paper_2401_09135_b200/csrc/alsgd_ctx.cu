// Host side of the C ABI: flat-buffer layout, arena carving, Algorithm 3's counter and boundary
// bookkeeping, worker dispatch state, and the translation of one ABI call into kernel launches.
#include "../../include/alsgd.h"
#include "alsgd_kernels.cuh"

#include <cmath>
#include <cstring>
#include <limits>
#include <new>
#include <vector>

using namespace alsgd;

namespace {

constexpr uint64_t kSliceAlign = 256;  // bytes; every arena slice starts on this boundary
constexpr int kStageChunks = 8;        // pieces a host gradient vector is copied in

enum WorkerState : uint8_t { kNever = 0, kDispatched = 1, kArrived = 2 };

struct Worker {
    float* p = nullptr;
    float* base = nullptr;       // the snapshot slot this worker was dispatched with (may be shared)
    int slot = -1;
    float* am = nullptr;
    float* av = nullptr;
    uint16_t* rep = nullptr;
    uint64_t pull_tick = 0;
    WorkerState state = kNever;
    // Right after a dispatch the worker's parameters equal its snapshot.  With snapshots in use the
    // copy into p is not made: readers take the snapshot instead until something writes p.
    bool p_in_snapshot = false;
};

uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

struct Carver {
    uint8_t* basep;
    uint64_t off = 0;
    explicit Carver(void* b) : basep(static_cast<uint8_t*>(b)) {}
    template <typename T>
    T* take(uint64_t count) {
        off = round_up(off, kSliceAlign);
        T* r = basep ? reinterpret_cast<T*>(basep + off) : nullptr;
        off += count * sizeof(T);
        return r;
    }
};

struct Segments {
    std::vector<uint64_t> end;
    std::vector<uint32_t> decay;
};

// Flat offsets, padded total and the weight-decay segments of the flat vector: maximal runs of
// elements with the same flag; padding between tensors is never decayed.
bool build_layout(const alsgd_tensor_desc* t, uint32_t n, uint32_t align, uint64_t* P, uint64_t* offs, Segments* seg) {
    if (!t || n == 0 || align == 0) return false;
    const uint64_t lim = std::numeric_limits<uint64_t>::max() / 8;
    uint64_t cur = 0;
    auto push = [&](uint64_t end, uint32_t dec) {
        if (!seg) return;
        if (!seg->end.empty() && seg->decay.back() == dec) { seg->end.back() = end; return; }
        seg->end.push_back(end);
        seg->decay.push_back(dec);
    };
    for (uint32_t i = 0; i < n; ++i) {
        if (t[i].numel == 0 || t[i].numel > lim || cur > lim) return false;
        if (offs) offs[i] = cur;
        const uint64_t end = cur + t[i].numel;
        push(end, (t[i].flags & ALSGD_TENSOR_DECAY) ? 1u : 0u);
        cur = round_up(end, align);
        if (cur != end) push(cur, 0u);
    }
    if (cur > lim) return false;
    *P = cur;
    return true;
}

bool valid_cfg(const alsgd_config* c) {
    if (!c) return false;
    if (c->n_workers == 0 || c->N == 0) return false;
    if (c->pg_base != ALSGD_PG_DISPATCH && c->pg_base != ALSGD_PG_CURRENT) return false;
    if (c->flags & ~(ALSGD_CFG_REPLICA_BF16 | ALSGD_CFG_GRAD_STAGING | ALSGD_CFG_OUTER_BUFFERED | ALSGD_CFG_OUTER_SGDM |
                     ALSGD_CFG_STABLE_PTRS)) return false;
    if ((c->flags & ALSGD_CFG_OUTER_BUFFERED) && (c->flags & ALSGD_CFG_OUTER_SGDM)) return false;
    if (!(c->beta >= 0.0f && c->beta < 1.0f)) return false;
    if (!std::isfinite(c->outer_lr)) return false;
    if (!(c->c >= 0.0f && (double)c->c * (double)c->N <= 1.0 + 1e-6)) return false;
    if (!(c->adam_b1 >= 0.0f && c->adam_b1 < 1.0f && c->adam_b2 >= 0.0f && c->adam_b2 < 1.0f)) return false;
    if (!(c->adam_eps >= 0.0f) || !(c->adam_wd >= 0.0f)) return false;
    return true;
}

}  // namespace

struct alsgd_ctx {
    alsgd_config cfg;
    uint64_t P = 0;
    cudaStream_t stream = nullptr;
    // device slices
    uint64_t* seg_end = nullptr;
    uint32_t* seg_decay = nullptr;
    uint32_t n_seg = 0;
    double* gnorm2 = nullptr;
    double* diag_partial = nullptr;
    unsigned int* nonfinite = nullptr;      // [0, 8): flags the pass ORs into; [8, 16): flags handed out; [16, 24): tickets
    unsigned int* guard_word = nullptr;   // debug build: violations recorded by the kernels' bounds checks
    float* theta = nullptr;
    float* mom = nullptr;
    float* delta = nullptr;
    float* grad_stage = nullptr;
    // Host gradients are copied in chunks on a stream of their own so that the step on chunk i runs while
    // chunk i+1 is still crossing PCIe.
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t stage_free = nullptr;               // main stream no longer reads the staging buffer
    cudaEvent_t chunk_ready[kStageChunks] = {};
    std::vector<Worker> workers;
    // Dispatch snapshots: W slots of P floats.  Workers dispatched together (one grace window, one
    // theta) share one slot, so the snapshot is written once per window and read once per batch.
    std::vector<float*> slot_ptr;
    std::vector<uint32_t> slot_ref;
    // Algorithm 3 bookkeeping
    uint64_t t = 0;
    bool delta_zero = true;     // Delta is zero by definition (start, or right after a boundary)
    bool delta_stored = true;   // ... and the arena really holds those zeros
    // scalars of Algorithm 3, each rounded to fp32 once
    float inv_n = 0, cb = 0, cn = 0;
    int last_cuda = 0;
    // Set when a call failed after some of its launches were already enqueued: the device state is then
    // ahead of the host bookkeeping, and every later state-changing call is refused.
    bool poisoned = false;
    // Consecutive whole-vector launches walk the vector in opposite directions, so that what the previous launch
    // touched last (and the L2 still holds) is what the next one touches first.
    uint32_t direction = 0;
    uintptr_t arena_lo = 0, arena_hi = 0;
};

namespace {

// Carve the arena; with arena == nullptr only the size is computed.
uint64_t carve(alsgd_ctx* c, void* arena, uint64_t P, const alsgd_config& cfg, uint32_t n_seg) {
    Carver k(arena);
    uint64_t* seg_end = k.take<uint64_t>(n_seg);
    uint32_t* seg_decay = k.take<uint32_t>(n_seg);
    double* gn = k.take<double>(kMaxArrivals);
    double* gpart = k.take<double>(diag_partial_count(P));
    unsigned int* nf = k.take<unsigned int>(3 * kMaxArrivals);
    unsigned int* gw = k.take<unsigned int>(1);
    float* theta = k.take<float>(P);
    float* mom = k.take<float>(P);
    float* delta = k.take<float>(P);
    if (c) {
        c->seg_end = seg_end; c->seg_decay = seg_decay; c->gnorm2 = gn; c->diag_partial = gpart; c->nonfinite = nf; c->guard_word = gw;
        c->theta = theta; c->mom = mom; c->delta = delta;
        c->workers.assign(cfg.n_workers, Worker());
        c->slot_ptr.clear();
        c->slot_ref.clear();
    }
    for (uint32_t w = 0; w < cfg.n_workers; ++w) {
        float* p = k.take<float>(P);
        float* base = cfg.pg_base == ALSGD_PG_DISPATCH ? k.take<float>(P) : nullptr;
        float* am = k.take<float>(P);
        float* av = k.take<float>(P);
        uint16_t* rep = (cfg.flags & ALSGD_CFG_REPLICA_BF16) ? k.take<uint16_t>(P) : nullptr;
        if (c) {
            Worker& W = c->workers[w];
            W.p = p; W.base = base; W.am = am; W.av = av; W.rep = rep;
            if (base) { W.slot = (int)w; c->slot_ptr.push_back(base); c->slot_ref.push_back(1u); }
        }
    }
    float* stage = (cfg.flags & ALSGD_CFG_GRAD_STAGING) ? k.take<float>(P) : nullptr;
    if (c) c->grad_stage = stage;
    return round_up(k.off, kSliceAlign);
}

int cuda_fail(alsgd_ctx* c, cudaError_t e) {
    if (c) c->last_cuda = (int)e;
    return ALSGD_E_CUDA;
}

#define ALSGD_CUDA(ctx, call)                                   \
    do {                                                        \
        cudaError_t e__ = (call);                               \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__);   \
    } while (0)

// Makes the context's device current for the duration of one ABI call.
struct DeviceGuard {
    int prev = -1;
    int target = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) : target(dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        if (ok && prev >= 0 && prev != target) cudaSetDevice(prev);
    }
};

int copy_vec(alsgd_ctx* c, void* dst, const void* src, uint64_t bytes, bool host_side) {
    ALSGD_CUDA(c, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, c->stream));
    if (host_side) ALSGD_CUDA(c, cudaStreamSynchronize(c->stream));
    return ALSGD_OK;
}

// Re-seed target: the worker's parameters and replica, plus (for one worker of the window) the
// snapshot slot the whole window will share.
void release_host_resources(alsgd_ctx* c) {
    if (c->copy_stream) { cudaStreamSynchronize(c->copy_stream); cudaStreamDestroy(c->copy_stream); c->copy_stream = nullptr; }
    if (c->stage_free) { cudaEventDestroy(c->stage_free); c->stage_free = nullptr; }
    for (int i = 0; i < kStageChunks; ++i)
        if (c->chunk_ready[i]) { cudaEventDestroy(c->chunk_ready[i]); c->chunk_ready[i] = nullptr; }
}

bool stable_ptrs(const alsgd_ctx* c) { return (c->cfg.flags & ALSGD_CFG_STABLE_PTRS) != 0; }

// Re-seed target s of a launch.  Normally the window's snapshot is written once (by the first target that is
// handed it) and the parameters are not stored at all: readers take the snapshot until something writes p.
// With ALSGD_CFG_STABLE_PTRS every worker keeps its own snapshot slot and its parameters are written too.
void fill_seed(const alsgd_ctx* c, ArriveArgs& a, uint32_t s, uint32_t worker, float* snapshot) {
    const Worker& w = c->workers[worker];
    const bool have_snapshots = !c->slot_ptr.empty();
    if (stable_ptrs(c)) {
        a.seed_p[s] = w.p;
        a.seed_base[s] = have_snapshots ? c->slot_ptr[worker] : nullptr;
    } else {
        a.seed_p[s] = have_snapshots ? nullptr : w.p;
        a.seed_base[s] = snapshot;
    }
    a.seed_rep[s] = w.rep;
}

void fill_guard(const alsgd_ctx* c, DebugGuard& g) {
#ifdef ALSGD_DEBUG_BOUNDS
    g.lo = c->arena_lo;
    g.hi = c->arena_hi;
    g.err = c->guard_word;
#else
    (void)c; (void)g;
#endif
}

// Where the worker's current parameters are to be read from.
const float* params_of(const Worker& w) { return w.p_in_snapshot ? w.base : w.p; }

// Make w.p hold the worker's parameters before handing the pointer out or copying from it.
int materialize_params(alsgd_ctx* c, Worker& w) {
    if (!w.p_in_snapshot) return ALSGD_OK;
    if (cudaMemcpyAsync(w.p, w.base, sizeof(float) * c->P, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess) {
        c->last_cuda = (int)cudaGetLastError();
        return ALSGD_E_CUDA;
    }
    w.p_in_snapshot = false;
    return ALSGD_OK;
}

// The slot that is free once the given workers have let go of theirs (-1 when the pseudo-gradient
// is taken against the running theta and no snapshots exist).  At most W - k other workers hold a
// slot, so one of the W slots is always free.
int pick_slot(const alsgd_ctx* c, const uint32_t* ids, uint32_t k) {
    if (c->slot_ptr.empty() || stable_ptrs(c)) return -1;
    std::vector<uint32_t> ref(c->slot_ref);
    for (uint32_t j = 0; j < k; ++j) {
        const int s = c->workers[ids[j]].slot;
        if (s >= 0) --ref[s];
    }
    for (size_t s = 0; s < ref.size(); ++s)
        if (ref[s] == 0) return (int)s;
    return -1;
}

void commit_slot(alsgd_ctx* c, const uint32_t* ids, uint32_t k, int s) {
    if (s < 0) return;                                   // no snapshots, or every worker keeps its own
    for (uint32_t j = 0; j < k; ++j) {
        Worker& w = c->workers[ids[j]];
        if (w.slot >= 0) --c->slot_ref[w.slot];
        w.slot = s;
        w.base = c->slot_ptr[s];
        w.p_in_snapshot = true;
        ++c->slot_ref[s];
    }
}

}  // namespace

extern "C" {

const char* alsgd_strerror(int status) {
    switch (status) {
        case ALSGD_OK: return "ok";
        case ALSGD_E_ARG: return "invalid argument";
        case ALSGD_E_RANGE: return "index out of range";
        case ALSGD_E_STATE: return "call not allowed in this state";
        case ALSGD_E_CUDA: return "CUDA runtime error";
        case ALSGD_E_NOMEM: return "not enough memory";
        case ALSGD_E_UNSUPPORTED: return "unsupported";
        case ALSGD_E_BOUNDS: return "a kernel access fell outside the arena (debug build)";
        default: return "unknown status";
    }
}

int alsgd_layout_size(const alsgd_tensor_desc* tensors, uint32_t n, uint32_t align_elems,
                      uint64_t* P_out, uint64_t* offsets_out) {
    if (!P_out) return ALSGD_E_ARG;
    uint64_t P = 0;
    if (!build_layout(tensors, n, align_elems, &P, offsets_out, nullptr)) return ALSGD_E_ARG;
    *P_out = P;
    return ALSGD_OK;
}

int alsgd_arena_bytes(const alsgd_tensor_desc* tensors, uint32_t n, uint32_t align_elems,
                      const alsgd_config* cfg, uint64_t* bytes_out) {
    if (!bytes_out || !valid_cfg(cfg)) return ALSGD_E_ARG;
    uint64_t P = 0;
    Segments seg;
    if (!build_layout(tensors, n, align_elems, &P, nullptr, &seg)) return ALSGD_E_ARG;
    *bytes_out = carve(nullptr, nullptr, P, *cfg, (uint32_t)seg.end.size());
    return ALSGD_OK;
}

int alsgd_init(alsgd_ctx** out, const alsgd_tensor_desc* tensors, uint32_t n, uint32_t align_elems,
               const alsgd_config* cfg) {
    if (!out || !valid_cfg(cfg) || !cfg->arena) return ALSGD_E_ARG;
    if (reinterpret_cast<uintptr_t>(cfg->arena) % kSliceAlign) return ALSGD_E_ARG;
    uint64_t P = 0;
    Segments seg;
    if (!build_layout(tensors, n, align_elems, &P, nullptr, &seg)) return ALSGD_E_ARG;
    const uint64_t need = carve(nullptr, nullptr, P, *cfg, (uint32_t)seg.end.size());
    if (cfg->arena_bytes < need) return ALSGD_E_NOMEM;

    alsgd_ctx* c = new (std::nothrow) alsgd_ctx();
    if (!c) return ALSGD_E_NOMEM;
    c->cfg = *cfg;
    c->P = P;
    c->stream = static_cast<cudaStream_t>(cfg->stream);
    c->n_seg = (uint32_t)seg.end.size();
    carve(c, cfg->arena, P, *cfg, c->n_seg);
    c->arena_lo = reinterpret_cast<uintptr_t>(cfg->arena);
    c->arena_hi = c->arena_lo + cfg->arena_bytes;
    // Scalars of Algorithm 3: evaluated in double from the fp32 inputs, rounded to fp32 once.
    c->inv_n = 1.0f / (float)cfg->N;
    c->cb = (float)(((double)1.0 - (double)cfg->c * (double)cfg->N + (double)cfg->c) * (double)cfg->beta);
    c->cn = (float)((double)cfg->c * (double)cfg->beta);

    int rc = ALSGD_OK;
    {
        DeviceGuard g(cfg->device);
        cudaError_t e = g.ok ? cudaSuccess : cudaErrorInvalidDevice;
        if (e == cudaSuccess) e = cudaMemcpyAsync(c->seg_end, seg.end.data(), sizeof(uint64_t) * c->n_seg, cudaMemcpyHostToDevice, c->stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(c->seg_decay, seg.decay.data(), sizeof(uint32_t) * c->n_seg, cudaMemcpyHostToDevice, c->stream);
        // The segment tables live in pageable host vectors that die with this scope.
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(c->gnorm2, 0, sizeof(double) * kMaxArrivals, c->stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(c->nonfinite, 0, sizeof(unsigned int) * 3 * kMaxArrivals, c->stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(c->guard_word, 0, sizeof(unsigned int), c->stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(c->theta, 0, sizeof(float) * P, c->stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(c->mom, 0, sizeof(float) * P, c->stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(c->delta, 0, sizeof(float) * P, c->stream);
        for (Worker& w : c->workers) {
            if (e == cudaSuccess) e = cudaMemsetAsync(w.p, 0, sizeof(float) * P, c->stream);
            if (e == cudaSuccess && w.base) e = cudaMemsetAsync(w.base, 0, sizeof(float) * P, c->stream);
            if (e == cudaSuccess) e = cudaMemsetAsync(w.am, 0, sizeof(float) * P, c->stream);
            if (e == cudaSuccess) e = cudaMemsetAsync(w.av, 0, sizeof(float) * P, c->stream);
            if (e == cudaSuccess && w.rep) e = cudaMemsetAsync(w.rep, 0, sizeof(uint16_t) * P, c->stream);
        }
        if (e == cudaSuccess && c->grad_stage) {
            e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->stage_free, cudaEventDisableTiming);
            for (int i = 0; i < kStageChunks && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&c->chunk_ready[i], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) { c->last_cuda = (int)e; rc = ALSGD_E_CUDA; }
    }
    if (rc != ALSGD_OK) { release_host_resources(c); delete c; return rc; }
    *out = c;
    return ALSGD_OK;
}

int alsgd_destroy(alsgd_ctx* ctx) {
    if (ctx) {
        DeviceGuard g(ctx->cfg.device);
        release_host_resources(ctx);
    }
    delete ctx;
    return ALSGD_OK;
}

int alsgd_set_global(alsgd_ctx* c, const float* src, int src_is_device) {
    if (!c || !src) return ALSGD_E_ARG;
    DeviceGuard g(c->cfg.device);
    return copy_vec(c, c->theta, src, sizeof(float) * c->P, !src_is_device);
}

int alsgd_get_global(alsgd_ctx* c, float* dst, int dst_is_device) {
    if (!c || !dst) return ALSGD_E_ARG;
    DeviceGuard g(c->cfg.device);
    return copy_vec(c, dst, c->theta, sizeof(float) * c->P, !dst_is_device);
}

int alsgd_set_worker_params(alsgd_ctx* c, uint32_t worker, const float* src, int src_is_device) {
    if (!c || !src) return ALSGD_E_ARG;
    if (worker >= c->cfg.n_workers) return ALSGD_E_RANGE;
    DeviceGuard g(c->cfg.device);
    c->workers[worker].p_in_snapshot = false;            // overwritten in full
    return copy_vec(c, c->workers[worker].p, src, sizeof(float) * c->P, !src_is_device);
}

int alsgd_get_worker_params(alsgd_ctx* c, uint32_t worker, float* dst, int dst_is_device) {
    if (!c || !dst) return ALSGD_E_ARG;
    if (worker >= c->cfg.n_workers) return ALSGD_E_RANGE;
    DeviceGuard g(c->cfg.device);
    return copy_vec(c, dst, params_of(c->workers[worker]), sizeof(float) * c->P, !dst_is_device);
}

int alsgd_pull(alsgd_ctx* c, uint32_t worker) {
    if (!c) return ALSGD_E_ARG;
    if (worker >= c->cfg.n_workers) return ALSGD_E_RANGE;
    if (c->poisoned) return ALSGD_E_STATE;
    Worker& w = c->workers[worker];
    ArriveArgs a{};
    a.theta = c->theta;
    a.n = c->P;
    a.n_arr = 0;
    a.n_seed = 1;
    fill_guard(c, a.guard);
    a.reverse = (c->direction ^= 1u);
    const int slot = pick_slot(c, &worker, 1);
    fill_seed(c, a, 0, worker, slot >= 0 ? c->slot_ptr[slot] : nullptr);
    DeviceGuard g(c->cfg.device);
    ALSGD_CUDA(c, launch_arrive(a, false, false, false, c->stream));
    commit_slot(c, &worker, 1, slot);
    w.pull_tick = c->t;
    w.state = kDispatched;
    return ALSGD_OK;
}

}  // extern "C"

namespace {

int adamw_impl(alsgd_ctx* c, uint32_t worker, const void* grads, bool bf16, int grads_is_device, uint64_t step, float lr) {
    if (!c || !grads || step == 0) return ALSGD_E_ARG;
    if (worker >= c->cfg.n_workers) return ALSGD_E_RANGE;
    Worker& w = c->workers[worker];
    if (w.state == kNever || c->poisoned) return ALSGD_E_STATE;
    if (!grads_is_device && !c->grad_stage) return ALSGD_E_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(grads) % 16) return ALSGD_E_ARG;
    DeviceGuard g(c->cfg.device);
    AdamArgs a{};
    fill_guard(c, a.guard);
    a.rep = w.rep;
    a.seg_end = c->seg_end; a.seg_decay = c->seg_decay; a.n_seg = c->n_seg;
    a.b1 = c->cfg.adam_b1; a.b2 = c->cfg.adam_b2;
    a.omb1 = 1.0f - a.b1; a.omb2 = 1.0f - a.b2;
    // Bias corrections: 1 - beta^step in double, rounded to fp32 once.
    a.bc1 = (float)(1.0 - std::pow((double)a.b1, (double)step));
    a.bc2 = (float)(1.0 - std::pow((double)a.b2, (double)step));
    a.eps = c->cfg.adam_eps; a.lr = lr; a.wd = c->cfg.adam_wd;
    const float* p_src = params_of(w);
    const uint64_t esz = bf16 ? sizeof(uint16_t) : sizeof(float);
    // One launch over [lo, lo + len) with the gradients at gsrc (device).
    auto launch_range = [&](uint64_t lo, uint64_t len, const void* gsrc) -> cudaError_t {
        a.p = w.p + lo; a.p_src = p_src + lo; a.m = w.am + lo; a.v = w.av + lo;
        a.rep = w.rep ? w.rep + lo : nullptr;
        a.g = bf16 ? nullptr : static_cast<const float*>(gsrc);
        a.g16 = bf16 ? static_cast<const uint16_t*>(gsrc) : nullptr;
        a.n = len;
        a.seg_base = lo;
        return launch_adamw(a, grads_is_device != 0, c->stream);
    };
    if (grads_is_device) {
        a.reverse = (c->direction ^= 1u);
        ALSGD_CUDA(c, launch_range(0, c->P, grads));
    } else {
        // Chunked: copy chunk i on the copy stream, run the step on it on the context's stream as soon as
        // it has landed; the next chunk's copy overlaps that launch.
        const uint64_t per = round_up((c->P + kStageChunks - 1) / kStageChunks, 1024);
        ALSGD_CUDA(c, cudaEventRecord(c->stage_free, c->stream));          // earlier launches may still read the buffer
        ALSGD_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->stage_free, 0));
        uint8_t* stage = reinterpret_cast<uint8_t*>(c->grad_stage);
        const uint8_t* src = static_cast<const uint8_t*>(grads);
        int i = 0;
        for (uint64_t lo = 0; lo < c->P; lo += per, ++i) {
            const uint64_t len = (c->P - lo < per) ? c->P - lo : per;
            ALSGD_CUDA(c, cudaMemcpyAsync(stage + lo * esz, src + lo * esz, len * esz, cudaMemcpyHostToDevice, c->copy_stream));
            ALSGD_CUDA(c, cudaEventRecord(c->chunk_ready[i], c->copy_stream));
            ALSGD_CUDA(c, cudaStreamWaitEvent(c->stream, c->chunk_ready[i], 0));
            const cudaError_t le = launch_range(lo, len, stage + lo * esz);
            if (le != cudaSuccess) {
                if (i > 0) c->poisoned = true;            // earlier pieces of this step are already enqueued
                return cuda_fail(c, le);
            }
        }
    }
    w.p_in_snapshot = false;
    return ALSGD_OK;
}

}  // namespace

extern "C" {

int alsgd_inner_adamw(alsgd_ctx* c, uint32_t worker, const float* grads, int grads_is_device,
                      uint64_t step, float lr) {
    return adamw_impl(c, worker, grads, false, grads_is_device, step, lr);
}

int alsgd_inner_adamw_bf16(alsgd_ctx* c, uint32_t worker, const uint16_t* grads, int grads_is_device,
                           uint64_t step, float lr) {
    return adamw_impl(c, worker, grads, true, grads_is_device, step, lr);
}

}  // extern "C"

namespace {

struct ArrivalPlan {
    uint64_t tick = 0;       // Algorithm 3's t this arrival is applied at (or would have been)
    uint64_t staleness = 0;
    float weight = 1.0f;
    bool dropped = false;
};

int arrive_impl(alsgd_ctx* c, const uint32_t* ids, uint32_t k, uint32_t flags, const alsgd_arrive_opts* opts,
                alsgd_arrival_info* info) {
    if (!c) return ALSGD_E_ARG;
    if (flags & ~(ALSGD_ARRIVE_RESEED | ALSGD_ARRIVE_NORM | ALSGD_ARRIVE_NANCHECK)) return ALSGD_E_ARG;
    if (opts) {
        if (!(opts->dc_lambda >= 0.0f) || !std::isfinite(opts->dc_lambda)) return ALSGD_E_ARG;
        if (opts->staleness_rule > ALSGD_STALE_POLY_THRES) return ALSGD_E_ARG;
    }
    if (k == 0) return ALSGD_OK;
    if (!ids) return ALSGD_E_ARG;
    const uint32_t W = c->cfg.n_workers;
    if (k > W) return ALSGD_E_ARG;
    std::vector<uint8_t> seen(W, 0);
    for (uint32_t j = 0; j < k; ++j) {
        if (ids[j] >= W) return ALSGD_E_RANGE;
        if (seen[ids[j]]) return ALSGD_E_ARG;
        seen[ids[j]] = 1;
    }
    for (uint32_t j = 0; j < k; ++j)
        if (c->workers[ids[j]].state != kDispatched) return ALSGD_E_STATE;
    if (c->poisoned) return ALSGD_E_STATE;

    const bool diag = (flags & (ALSGD_ARRIVE_NORM | ALSGD_ARRIVE_NANCHECK)) != 0;
    const bool reseed = (flags & ALSGD_ARRIVE_RESEED) != 0;
    const bool current = c->cfg.pg_base == ALSGD_PG_CURRENT;
    const bool sgdm = (c->cfg.flags & ALSGD_CFG_OUTER_SGDM) != 0;
    const bool buffered = sgdm || (c->cfg.flags & ALSGD_CFG_OUTER_BUFFERED) != 0;
    const bool stable = stable_ptrs(c);
    const uint32_t N = c->cfg.N;
    const uint32_t rule = opts ? opts->staleness_rule : ALSGD_STALE_NONE;
    const float dc_lambda = opts ? opts->dc_lambda : 0.0f;

    // ---- host plan: ticks, staleness, weights, discarded updates (Section 4, Poly / PolyThres)
    std::vector<ArrivalPlan> plan(k);
    std::vector<uint32_t> active;      // indices into ids[] of the arrivals that reach the kernel
    uint64_t t = c->t;
    bool extended = buffered || dc_lambda != 0.0f;
    for (uint32_t j = 0; j < k; ++j) {
        ArrivalPlan& a = plan[j];
        a.tick = t;
        a.staleness = t - c->workers[ids[j]].pull_tick;
        if (rule == ALSGD_STALE_POLY_THRES && a.staleness > opts->stale_threshold) { a.dropped = true; continue; }
        if (rule != ALSGD_STALE_NONE) a.weight = (float)std::pow(1.0 + (double)a.staleness, -0.5);
        else if (opts && opts->weights) a.weight = opts->weights[j];
        if (!std::isfinite(a.weight)) return ALSGD_E_ARG;
        if (a.weight != 1.0f) extended = true;
        active.push_back(j);
        ++t;
    }
    const uint32_t ka = (uint32_t)active.size();
    DeviceGuard g(c->cfg.device);

    // Everything below only enqueues; the bookkeeping is committed after the last launch succeeded.
    bool delta_zero = c->delta_zero, delta_stored = c->delta_stored;
    std::vector<double> norms(k, 0.0);
    std::vector<unsigned int> bads(k, 0u);

    const uint32_t n_chunks = (ka + kMaxArrivals - 1) / kMaxArrivals;
    uint32_t seeded = 0;  // how many of the last ids[] the final arrival launch re-seeds itself
    const int new_slot = reseed ? pick_slot(c, ids, k) : -1;   // one snapshot for the whole window
    float* snapshot = new_slot >= 0 ? c->slot_ptr[new_slot] : nullptr;
    bool snapshot_written = false;
    bool enqueued = false;       // a launch of this call is already on the stream
    // A failure after the first launch leaves theta, Delta and m ahead of the bookkeeping: refuse later calls.
    auto fail = [&](cudaError_t e) { if (enqueued) c->poisoned = true; return cuda_fail(c, e); };
#define ALSGD_STEP(call)                                 \
    do {                                                 \
        cudaError_t e__ = (call);                        \
        if (e__ != cudaSuccess) return fail(e__);        \
    } while (0)
    for (uint32_t ch = 0; ch < n_chunks; ++ch) {
        const uint32_t j0 = ch * kMaxArrivals;
        const uint32_t kk = (ka - j0 < (uint32_t)kMaxArrivals) ? ka - j0 : (uint32_t)kMaxArrivals;
        ArriveArgs a{};
        a.theta = c->theta; a.delta = c->delta; a.mom = c->mom;
        a.gnorm2 = c->gnorm2; a.diag_partial = c->diag_partial; a.nonfinite = c->nonfinite;
        a.nonfinite_out = c->nonfinite + kMaxArrivals; a.diag_ticket = c->nonfinite + 2 * kMaxArrivals;
        a.n = c->P;
        a.n_arr = kk;
        a.beta = c->cfg.beta; a.eps = c->cfg.outer_lr; a.inv_n = c->inv_n; a.cb = c->cb; a.cn = c->cn;
        a.dc_lambda = dc_lambda;
        // weights of the buffered step: Eq. 4 (beta^2, 1 + beta) or SGD Momentum (beta, 1)
        a.beta2 = sgdm ? c->cfg.beta : c->cfg.beta * c->cfg.beta;
        a.one_plus_beta = sgdm ? 1.0f : 1.0f + c->cfg.beta;
        fill_guard(c, a.guard);
        a.reverse = (c->direction ^= 1u);
        bool any_boundary = false, last_boundary = false;
        a.shared_base = current ? 0u : 1u;
        for (uint32_t j = 0; j < kk; ++j) {
            const uint32_t src = active[j0 + j];
            const Worker& w = c->workers[ids[src]];
            a.p[j] = params_of(w);
            a.base[j] = w.base;
            if (a.base[j] != a.base[0]) a.shared_base = 0u;
            a.w[j] = plan[src].weight;
            const bool b = ((plan[src].tick + 1) % N) == 0;          // Algorithm 3's boundary test
            if (b) { a.boundary_mask |= 1u << j; any_boundary = true; }
            last_boundary = b;
        }
        for (uint32_t j = kk; j < (uint32_t)kMaxArrivals; ++j) a.w[j] = 1.0f;
        if (delta_zero) a.flags |= kDeltaZeroIn;
        if (last_boundary && !stable) a.flags |= kDeltaSkipStore;
        if (buffered) {
            a.flags |= kBuffered;
            if (!any_boundary) a.flags |= kSkipThetaStore;
        } else if (c->cfg.c != 0.0f) {
            a.flags |= kCNonZero | kReadM;
        }
        if (dc_lambda != 0.0f) a.flags |= kDelayComp;
        if (any_boundary) a.flags |= kReadM | kWriteM;
        if (reseed && ch + 1 == n_chunks) {               // the final theta exists only in the last pass
            const uint32_t ns = k < (uint32_t)kMaxSeeds ? k : (uint32_t)kMaxSeeds;
            for (uint32_t s = 0; s < ns; ++s) fill_seed(c, a, s, ids[k - ns + s], s == 0 ? snapshot : nullptr);
            a.n_seed = ns;
            seeded = ns;
            snapshot_written = true;
        }
        ALSGD_STEP(launch_arrive(a, current, diag, extended, c->stream));
        enqueued = true;
        if (diag && info) {
            double nb[kMaxArrivals];
            unsigned int fb[kMaxArrivals];
            ALSGD_STEP(cudaMemcpyAsync(nb, c->gnorm2, sizeof(double) * kk, cudaMemcpyDeviceToHost, c->stream));
            ALSGD_STEP(cudaMemcpyAsync(fb, c->nonfinite + kMaxArrivals, sizeof(unsigned int) * kk, cudaMemcpyDeviceToHost, c->stream));
            ALSGD_STEP(cudaStreamSynchronize(c->stream));
            for (uint32_t j = 0; j < kk; ++j) { norms[active[j0 + j]] = nb[j]; bads[active[j0 + j]] = fb[j]; }
        }
        delta_zero = last_boundary;
        delta_stored = !last_boundary || stable;
    }
    // Workers the arrival launches did not re-seed (a batch larger than one launch, or nothing but
    // discarded updates): the same final theta through standalone pulls.
    if (reseed && seeded < k) {
        uint32_t left = k - seeded, at = 0;
        while (left) {
            const uint32_t ns = left < (uint32_t)kMaxSeeds ? left : (uint32_t)kMaxSeeds;
            ArriveArgs a{};
            a.theta = c->theta; a.n = c->P; a.n_seed = ns;
            fill_guard(c, a.guard);
            a.reverse = (c->direction ^= 1u);
            for (uint32_t s = 0; s < ns; ++s) {
                fill_seed(c, a, s, ids[at + s], snapshot_written ? nullptr : snapshot);
                snapshot_written = true;
            }
            ALSGD_STEP(launch_arrive(a, false, false, false, c->stream));
            enqueued = true;
            at += ns; left -= ns;
        }
    }
#undef ALSGD_STEP

    // ---- commit bookkeeping
    if (info) {
        for (uint32_t j = 0; j < k; ++j) {
            alsgd_arrival_info& o = info[j];
            o.tick = plan[j].tick;
            o.staleness = plan[j].staleness;
            o.worker = ids[j];
            o.dropped = plan[j].dropped ? 1u : 0u;
            o.boundary = (!plan[j].dropped && ((plan[j].tick + 1) % N) == 0) ? 1u : 0u;
            o.gnorm2 = (flags & ALSGD_ARRIVE_NORM) ? norms[j] : 0.0;
            o.nonfinite = (flags & ALSGD_ARRIVE_NANCHECK) ? (bads[j] ? 1u : 0u) : 0u;
        }
    }
    c->t = t;
    c->delta_zero = delta_zero;
    c->delta_stored = delta_stored;
    if (reseed) commit_slot(c, ids, k, new_slot);
    for (uint32_t j = 0; j < k; ++j) {
        Worker& w = c->workers[ids[j]];
        if (reseed) { w.state = kDispatched; w.pull_tick = c->t; }
        else w.state = kArrived;
    }
    return ALSGD_OK;
}

}  // namespace

extern "C" {

int alsgd_arrive(alsgd_ctx* c, const uint32_t* ids, uint32_t k, uint32_t flags, alsgd_arrival_info* info) {
    return arrive_impl(c, ids, k, flags, nullptr, info);
}

int alsgd_arrive_ex(alsgd_ctx* c, const uint32_t* ids, uint32_t k, uint32_t flags, const alsgd_arrive_opts* opts,
                    alsgd_arrival_info* info) {
    return arrive_impl(c, ids, k, flags, opts, info);
}

int alsgd_counters(alsgd_ctx* c, uint64_t* t_out, uint32_t* phase_out) {
    if (!c) return ALSGD_E_ARG;
    if (t_out) *t_out = c->t;
    if (phase_out) *phase_out = (uint32_t)(c->t % c->cfg.N);
    return ALSGD_OK;
}

int alsgd_state_ptrs(alsgd_ctx* c, alsgd_ptrs* out) {
    if (!c || !out) return ALSGD_E_ARG;
    if (c->delta_zero && !c->delta_stored) {
        DeviceGuard g(c->cfg.device);
        ALSGD_CUDA(c, cudaMemsetAsync(c->delta, 0, sizeof(float) * c->P, c->stream));
        c->delta_stored = true;
    }
    out->theta = c->theta; out->m = c->mom; out->delta = c->delta;
    out->P = c->P; out->n_workers = c->cfg.n_workers; out->reserved = 0;
    return ALSGD_OK;
}

int alsgd_worker_state_ptrs(alsgd_ctx* c, uint32_t worker, alsgd_worker_ptrs* out) {
    if (!c || !out) return ALSGD_E_ARG;
    if (worker >= c->cfg.n_workers) return ALSGD_E_RANGE;
    Worker& w = c->workers[worker];
    {
        DeviceGuard g(c->cfg.device);
        const int rc = materialize_params(c, w);
        if (rc != ALSGD_OK) return rc;
    }
    out->p = w.p; out->base = w.base; out->adam_m = w.am; out->adam_v = w.av; out->replica = w.rep;
    return ALSGD_OK;
}

}  // extern "C"

namespace {

struct ImageHeader {
    char magic[8];
    uint32_t version;
    uint32_t n_workers;
    uint64_t P;
    uint32_t N;
    uint32_t pg_base;
    uint32_t has_replica;
    uint32_t delta_zero;
    uint64_t t;
};
struct ImageWorker {
    uint64_t pull_tick;
    uint32_t state;
    uint32_t reserved;
};
const char kMagic[8] = {'A', 'L', 'S', 'G', 'D', 'C', 'K', '1'};

uint64_t image_bytes(const alsgd_ctx* c) {
    const uint64_t P = c->P;
    uint64_t per_worker = 3 * 4 * P;                               // p, adam m, adam v
    if (c->workers[0].base) per_worker += 4 * P;
    if (c->workers[0].rep) per_worker += 2 * P;
    return sizeof(ImageHeader) + sizeof(ImageWorker) * c->cfg.n_workers + 3 * 4 * P + per_worker * c->cfg.n_workers;
}

// Visit every device slice in image order.
template <typename F>
int for_each_slice(alsgd_ctx* c, F f) {
    const uint64_t P = c->P;
    int rc;
    if ((rc = f(c->theta, 4 * P)) || (rc = f(c->mom, 4 * P)) || (rc = f(c->delta, 4 * P))) return rc;
    for (Worker& w : c->workers) {
        if ((rc = f(w.p, 4 * P))) return rc;
        if (w.base && (rc = f(w.base, 4 * P))) return rc;
        if ((rc = f(w.am, 4 * P)) || (rc = f(w.av, 4 * P))) return rc;
        if (w.rep && (rc = f(w.rep, 2 * P))) return rc;
    }
    return ALSGD_OK;
}

}  // namespace

extern "C" {

int alsgd_state_bytes(alsgd_ctx* c, uint64_t* bytes_out) {
    if (!c || !bytes_out) return ALSGD_E_ARG;
    *bytes_out = image_bytes(c);
    return ALSGD_OK;
}

int alsgd_export_state(alsgd_ctx* c, void* host_dst, uint64_t bytes) {
    if (!c || !host_dst) return ALSGD_E_ARG;
    if (bytes < image_bytes(c)) return ALSGD_E_NOMEM;
    DeviceGuard g(c->cfg.device);
    if (c->delta_zero && !c->delta_stored) {                       // write out the zeros Delta stands for
        ALSGD_CUDA(c, cudaMemsetAsync(c->delta, 0, sizeof(float) * c->P, c->stream));
        c->delta_stored = true;
    }
    for (Worker& w : c->workers) {
        const int rc = materialize_params(c, w);
        if (rc != ALSGD_OK) return rc;
    }
    uint8_t* out = static_cast<uint8_t*>(host_dst);
    ImageHeader h{};
    std::memcpy(h.magic, kMagic, 8);
    h.version = 1; h.n_workers = c->cfg.n_workers; h.P = c->P; h.N = c->cfg.N; h.pg_base = c->cfg.pg_base;
    h.has_replica = c->workers[0].rep ? 1u : 0u; h.delta_zero = c->delta_zero ? 1u : 0u; h.t = c->t;
    std::memcpy(out, &h, sizeof(h));
    out += sizeof(h);
    for (const Worker& w : c->workers) {
        ImageWorker iw{w.pull_tick, (uint32_t)w.state, 0u};
        std::memcpy(out, &iw, sizeof(iw));
        out += sizeof(iw);
    }
    int rc = for_each_slice(c, [&](void* dev, uint64_t n) -> int {
        if (cudaMemcpyAsync(out, dev, n, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess) return cuda_fail(c, cudaGetLastError());
        out += n;
        return ALSGD_OK;
    });
    if (rc != ALSGD_OK) return rc;
    ALSGD_CUDA(c, cudaStreamSynchronize(c->stream));
    return ALSGD_OK;
}

int alsgd_import_state(alsgd_ctx* c, const void* host_src, uint64_t bytes) {
    if (!c || !host_src) return ALSGD_E_ARG;
    if (bytes < sizeof(ImageHeader)) return ALSGD_E_ARG;
    const uint8_t* in = static_cast<const uint8_t*>(host_src);
    ImageHeader h;
    std::memcpy(&h, in, sizeof(h));
    if (std::memcmp(h.magic, kMagic, 8) != 0 || h.version != 1) return ALSGD_E_ARG;
    if (h.P != c->P || h.n_workers != c->cfg.n_workers || h.N != c->cfg.N || h.pg_base != c->cfg.pg_base ||
        h.has_replica != (c->workers[0].rep ? 1u : 0u)) return ALSGD_E_ARG;
    if (bytes < image_bytes(c)) return ALSGD_E_ARG;
    in += sizeof(h);
    std::vector<ImageWorker> iw(c->cfg.n_workers);
    std::memcpy(iw.data(), in, sizeof(ImageWorker) * iw.size());
    for (const ImageWorker& w : iw)
        if (w.state > (uint32_t)kArrived) return ALSGD_E_ARG;
    in += sizeof(ImageWorker) * iw.size();
    DeviceGuard g(c->cfg.device);
    for (uint32_t w = 0; w < c->cfg.n_workers && !c->slot_ptr.empty(); ++w) {   // the image holds one snapshot per worker
        c->workers[w].slot = (int)w;
        c->workers[w].base = c->slot_ptr[w];
        c->slot_ref[w] = 1u;
    }
    for (Worker& w : c->workers) w.p_in_snapshot = false;       // the image carries the parameters themselves
    int rc = for_each_slice(c, [&](void* dev, uint64_t n) -> int {
        if (cudaMemcpyAsync(dev, in, n, cudaMemcpyHostToDevice, c->stream) != cudaSuccess) return cuda_fail(c, cudaGetLastError());
        in += n;
        return ALSGD_OK;
    });
    if (rc != ALSGD_OK) return rc;
    ALSGD_CUDA(c, cudaStreamSynchronize(c->stream));
    c->t = h.t;
    c->delta_zero = h.delta_zero != 0;
    c->delta_stored = true;
    c->poisoned = false;                                        // the whole state was replaced
    for (uint32_t w = 0; w < c->cfg.n_workers; ++w) {
        c->workers[w].pull_tick = iw[w].pull_tick;
        c->workers[w].state = (WorkerState)iw[w].state;
    }
    return ALSGD_OK;
}

int alsgd_sync(alsgd_ctx* c) {
    if (!c) return ALSGD_E_ARG;
    DeviceGuard g(c->cfg.device);
    ALSGD_CUDA(c, cudaStreamSynchronize(c->stream));
#ifdef ALSGD_DEBUG_BOUNDS
    unsigned int word = 0;
    ALSGD_CUDA(c, cudaMemcpyAsync(&word, c->guard_word, sizeof(word), cudaMemcpyDeviceToHost, c->stream));
    ALSGD_CUDA(c, cudaStreamSynchronize(c->stream));
    if (word) return ALSGD_E_BOUNDS;
#endif
    return ALSGD_OK;
}

int alsgd_debug_guard_limit(alsgd_ctx* c, uint64_t bytes) {
    if (!c) return ALSGD_E_ARG;
#ifdef ALSGD_DEBUG_BOUNDS
    const uint64_t whole = c->cfg.arena_bytes;
    if (bytes > whole) return ALSGD_E_ARG;
    c->arena_hi = c->arena_lo + (bytes ? bytes : whole);
    return ALSGD_OK;
#else
    (void)bytes;
    return ALSGD_E_UNSUPPORTED;
#endif
}

int alsgd_debug_word_ptr(alsgd_ctx* c, uint32_t** word_out) {
    if (!c || !word_out) return ALSGD_E_ARG;
#ifdef ALSGD_DEBUG_BOUNDS
    *word_out = c->guard_word;
    return ALSGD_OK;
#else
    *word_out = nullptr;
    return ALSGD_E_UNSUPPORTED;
#endif
}

int alsgd_last_cuda_error(alsgd_ctx* c) { return c ? c->last_cuda : 0; }

}  // extern "C"

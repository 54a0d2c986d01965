// Internal launch interface between the host-side context and the sm_100a kernels.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace alsgd {

constexpr int kMaxArrivals = 8;  // arrivals folded into one pass over theta / Delta / m
constexpr int kMaxSeeds = 8;     // replicas re-seeded by one launch

enum : uint32_t {
    kDeltaZeroIn = 1u,     // Delta is zero by definition on entry: do not read it
    kDeltaSkipStore = 2u,  // Delta is zero by definition on exit: do not write it
    kReadM = 4u,           // momentum is needed (a boundary in the batch, or c != 0)
    kWriteM = 8u,          // momentum changes (a boundary in the batch)
    kCNonZero = 16u,       // momentum activation c != 0
    kDelayComp = 32u,      // delay compensation on the pseudo-gradient (dc_lambda != 0)
    kBuffered = 64u,       // buffered outer step: theta and m move only at a boundary, by Eq. 4 on Delta/N
    kSkipThetaStore = 128u // theta is unchanged by this launch (buffered, no boundary): do not write it
};

// Debug build only (-DALSGD_DEBUG_BOUNDS): the byte range every arena-owned access must stay in and the
// word that records violations.  Empty in the normal build.
#ifdef ALSGD_DEBUG_BOUNDS
struct DebugGuard {
    uintptr_t lo = 0, hi = 0;   // [lo, hi): the arena
    unsigned int* err = nullptr;
};
#else
struct DebugGuard {};
#endif

// One batch of arrivals of Algorithm 3 plus the re-seed of the workers that are dispatched again.
struct ArriveArgs {
    float* theta;
    float* delta;
    float* mom;
    const float* base[kMaxArrivals];  // dispatch snapshots (unused when the pseudo-gradient is against running theta)
    const float* p[kMaxArrivals];     // arriving workers' parameters
    float* seed_p[kMaxSeeds];         // may be null (parameters are then read from the snapshot until first written)
    float* seed_base[kMaxSeeds];      // may be null
    uint16_t* seed_rep[kMaxSeeds];    // may be null
    double* gnorm2;                   // out: kMaxArrivals squared norms (written by the reduction that follows the pass)
    double* diag_partial;             // scratch: one double per block per arrival, diag_partial_count(n) entries
    unsigned int* nonfinite;          // scratch: kMaxArrivals flags the pass ORs into; zero on entry, put back to zero by the reduction
    unsigned int* nonfinite_out;      // out: kMaxArrivals flags (written by the reduction that follows the pass)
    unsigned int* diag_ticket;        // scratch: kMaxArrivals counters of the reduction; zero between launches
    uint64_t n;                       // elements
    uint32_t n_arr;
    uint32_t n_seed;
    uint32_t boundary_mask;           // bit j: arrival j is a momentum boundary
    uint32_t flags;
    float beta, eps, inv_n, cb, cn;
    // extended path only (weights, delay compensation, buffered outer step)
    float w[kMaxArrivals];            // staleness weights (1 = none)
    float dc_lambda;
    float beta2, one_plus_beta;       // momentum and gradient weights of the buffered step: beta*beta and 1+beta
                                      // (Eq. 4), or beta and 1 (SGD Momentum); each one fp32 operation
    uint32_t shared_base;             // 1: every arrival was dispatched with the snapshot base[0]
    uint32_t reverse;                 // 1: blocks take the tiles from the last to the first
    DebugGuard guard;
};

struct AdamArgs {
    float* p;                  // parameters out
    const float* p_src;        // parameters in (p itself, or the dispatch snapshot right after a dispatch)
    float* m;
    float* v;
    const float* g;            // fp32 gradients, or null when g16 is used
    const uint16_t* g16;       // bf16 gradients (bit patterns), or null
    uint16_t* rep;             // may be null
    const uint64_t* seg_end;   // device: ascending exclusive end of each weight-decay segment; last == n
    const uint32_t* seg_decay; // device: 1 if the segment is weight-decayed
    uint32_t n_seg;
    uint64_t n;                // elements in this launch
    uint64_t seg_base;         // flat index of this launch's first element (segment ends are flat indices)
    float b1, b2, omb1, omb2, bc1, bc2, eps, lr, wd;
    uint32_t reverse;          // 1: blocks take the tiles from the last to the first
    DebugGuard guard;
};

// Entries of ArriveArgs::diag_partial needed for a vector of n elements (any batch size).
uint64_t diag_partial_count(uint64_t n);

cudaError_t launch_arrive(const ArriveArgs& a, bool pg_current, bool diagnostics, bool extended, cudaStream_t s);
// dependent_launch: allow the kernel's blocks to be placed while the stream's previous kernel drains (off where
// the launch also waits on an event of another stream).
cudaError_t launch_adamw(const AdamArgs& a, bool dependent_launch, cudaStream_t s);

}  // namespace alsgd

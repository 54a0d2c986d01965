/*
 * alsgd_sweep.h — C ABI of the launch-shape benchmark library (libalsgd_sweep.so).
 *
 * Not part of the method: the paper says nothing about kernels.  This library holds many launch
 * shapes (threads per block, vectors per thread, minimum resident blocks, one tile per block or a
 * persistent grid-stride loop, scalar or packed two-lane arithmetic, per-arrival or shared dispatch
 * snapshot) of exactly the kernel bodies libalsgd.so runs, so that the choice of the shapes the
 * product uses can be re-measured at any time (bench.py --shape-sweep).  It does the real work of
 * the step on the buffers it is given; it keeps no state and allocates nothing.
 */
#ifndef ALSGD_SWEEP_H
#define ALSGD_SWEEP_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ALSGD_SWEEP_ADAMW 0u
#define ALSGD_SWEEP_ARRIVE 1u

typedef struct alsgd_sweep_variant {
    uint32_t kind;       /* ALSGD_SWEEP_ADAMW or ALSGD_SWEEP_ARRIVE */
    uint32_t K;          /* arrivals per pass (arrive only); all K workers are re-seeded in the same pass */
    uint32_t base_mode;  /* 0: one dispatch snapshot per arrival, 1: one shared by all, 2: running theta */
    uint32_t V;          /* float4 vectors per thread per stream */
    uint32_t block;      /* threads per block */
    uint32_t min_blocks; /* second argument of __launch_bounds__ (1 = unconstrained) */
    uint32_t persistent; /* 1: grid of resident blocks looping over tiles; 0: one tile per block */
    uint32_t packed;     /* 1: f32x2 two-lane arithmetic */
    uint32_t diag;       /* 1: with the squared-norm / non-finite diagnostics */
    uint32_t staged;     /* 0: operands move through registers (128-bit loads and stores); otherwise the tile size in
                            elements of a variant that moves every stream with 1-D bulk copies (cp.async.bulk global ->
                            shared with an mbarrier, arithmetic from shared memory, cp.async.bulk shared -> global) */
} alsgd_sweep_variant;

/* All pointers are device pointers to caller-owned buffers of n elements (16-byte aligned), except where noted. */
typedef struct alsgd_sweep_buffers {
    uint64_t n;
    float* theta;
    float* delta;
    float* mom;
    const float* p[8];        /* arriving workers' parameters */
    const float* base[8];     /* their dispatch snapshots (base[0] alone is read when base_mode = 1) */
    float* snapshot;          /* the window's new snapshot, written by the re-seed */
    uint16_t* rep[8];         /* bf16 replicas written by the re-seed */
    float* adam_p;
    float* adam_m;
    float* adam_v;
    const float* adam_g;
    uint16_t* adam_rep;
    const uint64_t* seg_end;  /* weight-decay segment table: n_seg ascending exclusive ends, last == n */
    const uint32_t* seg_decay;
    uint32_t n_seg;
    uint32_t reserved;
    double* diag_scratch;     /* 8 * (n / 256 + 66) doubles (diag variants only) */
    double* diag_out;         /* 8 doubles */
    unsigned int* diag_flags; /* 8 words, zero before the first launch */
    unsigned int* diag_state; /* 16 words, zero before the first launch: 8 counters of the reduction, then the 8 flags it hands out */
} alsgd_sweep_buffers;

/* Position in the Delayed Nesterov cycle an arrival pass is timed at. */
#define ALSGD_SWEEP_PHASE_MIDDLE 0u  /* Delta read and written, no momentum boundary in the batch */
#define ALSGD_SWEEP_PHASE_CYCLE 1u   /* the batch is a whole cycle (N = K): Delta neither read nor written, m read and written */

/* OR-ed into `phase`: launch as a programmatic dependent launch (the kernel's blocks may be placed while the previous
 * kernel of the stream drains and wait, before their first memory access, for its completion).  Register variants only. */
#define ALSGD_SWEEP_LAUNCH_DEPENDENT 0x100u

/* OR-ed into `phase` (AdamW variants): walk the vector in the opposite direction of the previous launch, so that the
 * state the previous launch touched last, which L2 still holds, is touched first. */
#define ALSGD_SWEEP_LAUNCH_ALTERNATE 0x200u

int alsgd_sweep_count(void);
/* idx in [0, count).  Returns 0, or -1 for a bad index or null pointer. */
int alsgd_sweep_describe(int idx, alsgd_sweep_variant* out);
/* Enqueue one launch of variant idx on the stream (cudaStream_t).  Returns 0 or the cudaError_t of the launch.
 * Staged variants need n to be a multiple of 8 and 16-byte aligned buffers (cudaErrorInvalidValue otherwise) and
 * record a wait that ran out in b->diag_flags[7] instead of hanging. */
int alsgd_sweep_launch(int idx, const alsgd_sweep_buffers* b, uint32_t phase, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ALSGD_SWEEP_H */

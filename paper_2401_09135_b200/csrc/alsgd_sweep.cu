// Launch-shape benchmark library: many instantiations of the kernel bodies of alsgd_kernels_impl.cuh behind
// the small C ABI of include/alsgd_sweep.h.  Built as its own shared library so that the product library
// carries only the shapes it runs.
#include "../../include/alsgd_sweep.h"
#include "alsgd_kernels_impl.cuh"

namespace {

using namespace alsgd;
using namespace alsgd::kern;

typedef cudaError_t (*LaunchFn)(const alsgd_sweep_buffers&, uint32_t, cudaStream_t);

struct Entry {
    alsgd_sweep_variant v;
    LaunchFn fn;
};

// Blocks of a persistent launch: every block the device can hold at once.
template <typename Kern>
unsigned resident_grid(Kern kern, int block, unsigned tiles) {
    int dev = 0, sms = 0, per_sm = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, block, 0);
    const unsigned g = (unsigned)(sms * (per_sm > 0 ? per_sm : 1));
    return g < tiles ? g : tiles;
}

template <int K, int V, int BLK, int MINB, bool DIAG, int BASE, bool PERSIST, bool PK>
cudaError_t run_arrive(const alsgd_sweep_buffers& b, uint32_t phase, cudaStream_t s) {
    ArriveArgs a{};
    a.theta = b.theta; a.delta = b.delta; a.mom = b.mom;
    a.n = b.n; a.n_arr = K; a.n_seed = K;
    for (int j = 0; j < K; ++j) {
        a.p[j] = b.p[j];
        a.base[j] = b.base[BASE == kBaseShared ? 0 : j];
        a.seed_rep[j] = b.rep[j];
    }
    for (int j = 0; j < kMaxArrivals; ++j) a.w[j] = 1.0f;
    a.seed_base[0] = b.snapshot;
    a.shared_base = BASE == kBaseShared;
    a.beta = 0.9f; a.eps = 0.7f; a.inv_n = 1.0f / (float)(K > 4 ? 8 : 4); a.cb = 0.9f; a.cn = 0.0f;
    if (phase == ALSGD_SWEEP_PHASE_CYCLE) {
        a.flags = kDeltaZeroIn | kDeltaSkipStore | kReadM | kWriteM;
        a.boundary_mask = 1u << (K - 1);
    }
    a.gnorm2 = b.diag_out; a.diag_partial = b.diag_scratch; a.nonfinite = b.diag_flags;
    auto kern = arrive_kernel<K, V, BLK, MINB, DIAG, BASE, false, PERSIST, PK>;
    unsigned grid = 1;
    cudaError_t e = grid_for(a.n, (uint64_t)V * BLK, &grid);
    if (e != cudaSuccess) return e;
    if (PERSIST) grid = resident_grid(kern, BLK, grid);
    kern<<<grid, BLK, 0, s>>>(a);
    if (DIAG) {
        double* chunk_sum = a.diag_partial + (uint64_t)K * grid;
        diag_reduce1_kernel<<<dim3(kDiagChunks, K), kDiagBlock, 0, s>>>(a.diag_partial, grid, chunk_sum);
        diag_reduce2_kernel<<<1, 32, 0, s>>>(chunk_sum, K, a.gnorm2);
    }
    return cudaGetLastError();
}

template <int V, int BLK, int MINB, bool PERSIST>
cudaError_t run_adamw(const alsgd_sweep_buffers& b, uint32_t, cudaStream_t s) {
    AdamArgs a{};
    a.p = b.adam_p; a.p_src = b.adam_p; a.m = b.adam_m; a.v = b.adam_v; a.g = b.adam_g; a.rep = b.adam_rep;
    a.seg_end = b.seg_end; a.seg_decay = b.seg_decay; a.n_seg = b.n_seg;
    a.n = b.n; a.seg_base = 0;
    a.b1 = 0.9f; a.b2 = 0.95f; a.omb1 = 1.0f - a.b1; a.omb2 = 1.0f - a.b2;
    a.bc1 = 0.65f; a.bc2 = 0.4f; a.eps = 1e-8f; a.lr = 1e-3f; a.wd = 0.1f;
    auto kern = adamw_kernel<V, BLK, MINB, false, PERSIST>;
    unsigned grid = 1;
    cudaError_t e = grid_for(a.n, (uint64_t)V * BLK, &grid);
    if (e != cudaSuccess) return e;
    if (PERSIST) grid = resident_grid(kern, BLK, grid);
    kern<<<grid, BLK, 0, s>>>(a);
    return cudaGetLastError();
}

#define ARR(K, V, BLK, MINB, DIAG, BASE, PERSIST, PK) \
    {{ALSGD_SWEEP_ARRIVE, K, BASE, V, BLK, MINB, PERSIST, PK, DIAG, 0}, &run_arrive<K, V, BLK, MINB, DIAG, BASE, PERSIST, PK>},
#define ADM(V, BLK, MINB, PERSIST) \
    {{ALSGD_SWEEP_ADAMW, 0, 0, V, BLK, MINB, PERSIST, 0, 0, 0}, &run_adamw<V, BLK, MINB, PERSIST>},

// one tile per block, scalar and packed arithmetic, over the block-size / vectors-per-thread grid
#define ARR_SHAPES(K, DIAG, BASE)                                           \
    ARR(K, 1, 64, 1, DIAG, BASE, 0, 0) ARR(K, 1, 64, 1, DIAG, BASE, 0, 1)   \
    ARR(K, 1, 128, 1, DIAG, BASE, 0, 0) ARR(K, 1, 128, 1, DIAG, BASE, 0, 1) \
    ARR(K, 1, 256, 1, DIAG, BASE, 0, 0) ARR(K, 1, 256, 1, DIAG, BASE, 0, 1) \
    ARR(K, 1, 512, 1, DIAG, BASE, 0, 0) ARR(K, 1, 512, 1, DIAG, BASE, 0, 1) \
    ARR(K, 2, 64, 1, DIAG, BASE, 0, 0) ARR(K, 2, 64, 1, DIAG, BASE, 0, 1)   \
    ARR(K, 2, 128, 1, DIAG, BASE, 0, 0) ARR(K, 2, 128, 1, DIAG, BASE, 0, 1) \
    ARR(K, 2, 256, 1, DIAG, BASE, 0, 0) ARR(K, 2, 256, 1, DIAG, BASE, 0, 1) \
    ARR(K, 4, 128, 1, DIAG, BASE, 0, 0) ARR(K, 4, 128, 1, DIAG, BASE, 0, 1) \
    ARR(K, 4, 256, 1, DIAG, BASE, 0, 0) ARR(K, 4, 256, 1, DIAG, BASE, 0, 1)
#define ARR_DIAG_SHAPES(K, BASE)                                      \
    ARR(K, 1, 64, 1, 1, BASE, 0, 0)                                   \
    ARR(K, 1, 128, 1, 1, BASE, 0, 0) ARR(K, 1, 128, 1, 1, BASE, 0, 1) \
    ARR(K, 1, 256, 1, 1, BASE, 0, 0) ARR(K, 1, 256, 1, 1, BASE, 0, 1) \
    ARR(K, 2, 128, 1, 1, BASE, 0, 0) ARR(K, 2, 256, 1, 1, BASE, 0, 0)

const Entry kEntries[] = {
    ADM(1, 64, 1, 0) ADM(1, 128, 1, 0) ADM(1, 256, 1, 0) ADM(1, 512, 1, 0) ADM(1, 1024, 1, 0)
    ADM(2, 64, 1, 0) ADM(2, 128, 1, 0) ADM(2, 256, 1, 0) ADM(2, 512, 1, 0)
    ADM(4, 128, 1, 0) ADM(4, 256, 1, 0)
    ADM(1, 256, 1, 1) ADM(2, 256, 1, 1) ADM(4, 256, 1, 1)
    ARR_SHAPES(1, 0, kBasePerArrival)
    ARR_SHAPES(2, 0, kBasePerArrival) ARR_SHAPES(2, 0, kBaseShared)
    ARR_SHAPES(4, 0, kBasePerArrival) ARR_SHAPES(4, 0, kBaseShared)
    ARR_SHAPES(8, 0, kBasePerArrival) ARR_SHAPES(8, 0, kBaseShared)
    ARR_DIAG_SHAPES(1, kBasePerArrival) ARR_DIAG_SHAPES(4, kBaseShared) ARR_DIAG_SHAPES(8, kBaseShared)
    ARR_DIAG_SHAPES(8, kBasePerArrival)
    // persistent grid-stride loops of the same bodies
    ARR(1, 1, 256, 1, 0, kBasePerArrival, 1, 0) ARR(1, 4, 256, 1, 0, kBasePerArrival, 1, 0)
    ARR(8, 1, 256, 1, 0, kBaseShared, 1, 0) ARR(8, 1, 128, 1, 0, kBaseShared, 1, 0)
    // register caps that force more resident blocks
    ARR(8, 1, 256, 3, 0, kBasePerArrival, 0, 0) ARR(8, 1, 256, 4, 0, kBasePerArrival, 0, 0)
    ARR(8, 1, 128, 6, 0, kBasePerArrival, 0, 0) ARR(8, 1, 128, 8, 0, kBasePerArrival, 0, 0)
    ARR(8, 1, 256, 4, 0, kBaseShared, 0, 0) ARR(8, 1, 128, 8, 0, kBaseShared, 0, 0)
    ARR(4, 2, 256, 3, 0, kBasePerArrival, 0, 0) ARR(4, 2, 256, 3, 0, kBaseShared, 0, 0)
    ARR(1, 4, 256, 3, 0, kBasePerArrival, 0, 0) ARR(1, 4, 128, 6, 0, kBasePerArrival, 0, 0)
    ARR(8, 1, 128, 6, 1, kBaseShared, 0, 0) ARR(8, 1, 128, 7, 1, kBaseShared, 0, 0)
    ARR(8, 1, 128, 5, 1, kBasePerArrival, 0, 0) ARR(8, 1, 64, 12, 1, kBaseShared, 0, 0)
};
constexpr int kCount = (int)(sizeof(kEntries) / sizeof(kEntries[0]));

}  // namespace

extern "C" {

int alsgd_sweep_count(void) { return kCount; }

int alsgd_sweep_describe(int idx, alsgd_sweep_variant* out) {
    if (idx < 0 || idx >= kCount || !out) return -1;
    *out = kEntries[idx].v;
    return 0;
}

int alsgd_sweep_launch(int idx, const alsgd_sweep_buffers* b, uint32_t phase, void* stream) {
    if (idx < 0 || idx >= kCount || !b || b->n == 0) return (int)cudaErrorInvalidValue;
    return (int)kEntries[idx].fn(*b, phase, static_cast<cudaStream_t>(stream));
}

}  // extern "C"

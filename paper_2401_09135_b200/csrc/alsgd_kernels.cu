// The launch shapes the library runs, and the dispatch from one ABI call's arguments to a kernel
// instantiation.  The kernel bodies are in alsgd_kernels_impl.cuh.
#include "alsgd_kernels_impl.cuh"

namespace alsgd {

namespace {

using namespace kern;

// Launch shape per number of arrivals K: float4 vectors per thread per stream, threads per block, packed
// two-lane arithmetic.  From the launch-shape benchmark (bench.py --shape-sweep) on B200 at 110M elements:
// every one-tile-per-block shape with at most ~20 vectors in flight per thread lands within 1 % of 6.8 TB/s
// (the memory system's rate for these read/write mixes); what separates them is how they degrade once the
// diagnostics or eight arrivals add registers and arithmetic.  One vector per thread keeps the registers low
// at every K (K = 8: 69-96 registers; two vectors per thread lose 2-10 %, four up to 40 %); with five or more
// arrivals 128-thread blocks fit more warps into the register file than 256-thread blocks (96 registers: five
// blocks of four warps against two of eight), worth about 0.5 %; at K <= 4 neither matters.
// Packed arithmetic stays off: it gains at most 1.3 % and is not bit-identical (see Lanes in the header).
struct Shape {
    int V, BLK;
    bool PK;
};
constexpr Shape arrive_shape(int K) {
    if (K == 0) return {4, 256, false};           // re-seed only: one read stream, up to three written
    if (K <= 4) return {1, 256, false};
    return {1, 128, false};
}
// AdamW with the 110M layout's weight-decay table (every thread looks its segment up once, so one vector per
// thread pays that latency twice as often): 2 x 128 6.79-6.82 TB/s, 2 x 64 6.79, 2 x 256 6.32-6.64, 1 x 128 6.47-6.51.
constexpr Shape kAdamShape = {2, 128, false};
constexpr int kMinTileVecs = 128;                 // smallest BLK * V of any arrival shape: the most blocks a launch can have

template <int K, bool DIAG, int BASE, bool EXT>
cudaError_t launch_arrive_k(const ArriveArgs& a, cudaStream_t s) {
    constexpr Shape sh = arrive_shape(K);
    static_assert(sh.V * sh.BLK >= kMinTileVecs, "diag_partial_count assumes at least kMinTileVecs vectors per block");
    // With the diagnostics the eight-arrival kernel on a shared snapshot needs 78 registers, one block per SM fewer
    // than the 72 that seven resident blocks of 128 threads allow; capping it there costs no spills and measured +1.2 %.
    constexpr int min_blocks = (DIAG && K >= 5 && BASE == kBaseShared) ? 7 : 1;
    auto kern = arrive_kernel<K, sh.V, sh.BLK, min_blocks, DIAG, BASE, EXT, false, sh.PK>;
    unsigned grid = 1;
    cudaError_t e = grid_for(a.n, (uint64_t)sh.V * sh.BLK, &grid);
    if (e != cudaSuccess) return e;
    // Programmatic dependent launch: the blocks may be placed while the stream's previous kernel drains (they wait
    // for its completion before their first access); at 23M elements this hides 1-2 % of launch gap, at 110M ~0.
    e = launch_kernel(kern, grid, sh.BLK, s, a, true);
    if (e != cudaSuccess) return e;
    if (DIAG && K > 0) {
        double* chunk_sum = a.diag_partial + (uint64_t)K * grid;        // behind the K x grid partials
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(kDiagChunks, K);
        cfg.blockDim = dim3(kDiagBlock);
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, diag_reduce_kernel, (const double*)a.diag_partial, (uint32_t)grid, chunk_sum, a.gnorm2,
                               a.nonfinite, a.nonfinite_out, a.diag_ticket);
        if (e != cudaSuccess) return e;
    }
    return cudaGetLastError();
}

template <bool DIAG, int BASE, bool EXT>
cudaError_t launch_arrive_n(const ArriveArgs& a, cudaStream_t s) {
    switch (a.n_arr) {
        case 1: return launch_arrive_k<1, DIAG, BASE, EXT>(a, s);
        case 2: return launch_arrive_k<2, DIAG, BASE, EXT>(a, s);
        case 3: return launch_arrive_k<3, DIAG, BASE, EXT>(a, s);
        case 4: return launch_arrive_k<4, DIAG, BASE, EXT>(a, s);
        case 5: return launch_arrive_k<5, DIAG, BASE, EXT>(a, s);
        case 6: return launch_arrive_k<6, DIAG, BASE, EXT>(a, s);
        case 7: return launch_arrive_k<7, DIAG, BASE, EXT>(a, s);
        case 8: return launch_arrive_k<8, DIAG, BASE, EXT>(a, s);
        default: return cudaErrorInvalidValue;
    }
}

template <bool DIAG, int BASE>
cudaError_t launch_arrive_e(const ArriveArgs& a, bool extended, cudaStream_t s) {
    return extended ? launch_arrive_n<DIAG, BASE, true>(a, s) : launch_arrive_n<DIAG, BASE, false>(a, s);
}

template <int BASE>
cudaError_t launch_arrive_d(const ArriveArgs& a, bool diagnostics, bool extended, cudaStream_t s) {
    return diagnostics ? launch_arrive_e<true, BASE>(a, extended, s) : launch_arrive_e<false, BASE>(a, extended, s);
}

}  // namespace

uint64_t diag_partial_count(uint64_t n) {
    const uint64_t blocks = ((n >> 2) + kMinTileVecs - 1) / kMinTileVecs + 1;
    return (blocks + kern::kDiagChunks) * kMaxArrivals;
}

cudaError_t launch_arrive(const ArriveArgs& a, bool pg_current, bool diagnostics, bool extended, cudaStream_t s) {
    if (a.n == 0) return cudaSuccess;
    if (a.n_arr > (uint32_t)kMaxArrivals || a.n_seed > (uint32_t)kMaxSeeds) return cudaErrorInvalidValue;
    if (a.n_arr == 0) return launch_arrive_k<0, false, kBaseCurrent, false>(a, s);      // re-seed only
    if (pg_current) return launch_arrive_d<kBaseCurrent>(a, diagnostics, extended, s);
    if (a.shared_base && a.n_arr > 1) return launch_arrive_d<kBaseShared>(a, diagnostics, extended, s);
    return launch_arrive_d<kBasePerArrival>(a, diagnostics, extended, s);
}

cudaError_t launch_adamw(const AdamArgs& a, bool dependent_launch, cudaStream_t s) {
    if (a.n == 0) return cudaSuccess;
    constexpr Shape sh = kAdamShape;
    unsigned grid = 1;
    cudaError_t e = grid_for(a.n, (uint64_t)sh.V * sh.BLK, &grid);
    if (e != cudaSuccess) return e;
    if (a.g16) return launch_kernel(adamw_kernel<sh.V, sh.BLK, 1, true, false>, grid, sh.BLK, s, a, dependent_launch);
    return launch_kernel(adamw_kernel<sh.V, sh.BLK, 1, false, false>, grid, sh.BLK, s, a, dependent_launch);
}

}  // namespace alsgd

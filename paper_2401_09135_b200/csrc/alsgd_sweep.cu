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
    const bool pdl = (phase & ALSGD_SWEEP_LAUNCH_DEPENDENT) != 0;
    phase &= ~ALSGD_SWEEP_LAUNCH_DEPENDENT;
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
    e = launch_kernel(kern, grid, BLK, s, a, pdl);
    if (e != cudaSuccess) return e;
    if (DIAG) {
        double* chunk_sum = a.diag_partial + (uint64_t)K * grid;
        diag_reduce_kernel<<<dim3(kDiagChunks, K), kDiagBlock, 0, s>>>(a.diag_partial, grid, chunk_sum, a.gnorm2, a.nonfinite,
                                                                       b.diag_state + 8, b.diag_state);
    }
    return cudaGetLastError();
}

template <int V, int BLK, int MINB, bool PERSIST>
cudaError_t run_adamw(const alsgd_sweep_buffers& b, uint32_t phase, cudaStream_t s) {
    AdamArgs a{};
    a.p = b.adam_p; a.p_src = b.adam_p; a.m = b.adam_m; a.v = b.adam_v; a.g = b.adam_g; a.rep = b.adam_rep;
    a.seg_end = b.seg_end; a.seg_decay = b.seg_decay; a.n_seg = b.n_seg;
    a.n = b.n; a.seg_base = 0;
    a.b1 = 0.9f; a.b2 = 0.95f; a.omb1 = 1.0f - a.b1; a.omb2 = 1.0f - a.b2;
    a.bc1 = 0.65f; a.bc2 = 0.4f; a.eps = 1e-8f; a.lr = 1e-3f; a.wd = 0.1f;
    static unsigned flip = 0;
    if (phase & ALSGD_SWEEP_LAUNCH_ALTERNATE) a.reverse = (flip++) & 1u;
    auto kern = adamw_kernel<V, BLK, MINB, false, PERSIST>;
    unsigned grid = 1;
    cudaError_t e = grid_for(a.n, (uint64_t)V * BLK, &grid);
    if (e != cudaSuccess) return e;
    if (PERSIST) grid = resident_grid(kern, BLK, grid);
    return launch_kernel(kern, grid, BLK, s, a, (phase & ALSGD_SWEEP_LAUNCH_DEPENDENT) != 0);
}

// ---------------------------------------------------------------------------------------------------------
// The AdamW stream with every operand moved by the copy engine instead of through registers: one tile per
// block; one thread starts four 1-D bulk copies global -> shared that complete on an mbarrier; all threads
// wait for it (bounded), do the arithmetic from shared memory in place, and one thread starts four bulk copies
// shared -> global.  Same arithmetic (adam_element) and the same bytes as adamw_kernel; benchmark only.
// Every copy starts on a 16-byte boundary and has a size that is a multiple of 16 bytes: tiles are multiples
// of 8 elements, and so is n (checked by the launcher).  No multicast, no cluster.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_addr(dst_smem)), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, const void* src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 :: "l"(dst), "r"(smem_addr(src_smem)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

constexpr int kWaitLimit = 1 << 22;     // polls of the mbarrier before a block gives up and records it

template <int TILE, int BLK>
__global__ void __launch_bounds__(BLK) adamw_bulk_kernel(const __grid_constant__ AdamArgs a, unsigned int* gave_up) {
    extern __shared__ __align__(128) unsigned char smem[];
    float* sg = reinterpret_cast<float*>(smem);
    float* sp = sg + TILE;
    float* sm = sp + TILE;
    float* sv = sm + TILE;
    uint16_t* srep = reinterpret_cast<uint16_t*>(sv + TILE);
    __shared__ __align__(8) unsigned long long bar_storage;
    const uint32_t bar = smem_addr(&bar_storage);
    const uint64_t t0 = (uint64_t)blockIdx.x * TILE;
    const uint32_t cnt = (uint32_t)(a.n - t0 < (uint64_t)TILE ? a.n - t0 : (uint64_t)TILE);   // multiple of 8
    const uint32_t bytes = cnt * 4u;

    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(1) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(4u * bytes) : "memory");
        bulk_load(sg, a.g + t0, bytes, bar);
        bulk_load(sp, a.p_src + t0, bytes, bar);
        bulk_load(sm, a.m + t0, bytes, bar);
        bulk_load(sv, a.v + t0, bytes, bar);
    }
    bool landed = false;
    for (int it = 0; it < kWaitLimit && !landed; ++it) landed = mbar_try_wait(bar, 0);
    // The block decides together (a completed phase stays completed, so one thread that saw it is proof), and
    // either every thread goes on or every thread leaves: nobody is left waiting at a barrier.
    if (!__syncthreads_or(landed)) {                 // record it, give the copies one more bounded wait, leave
        if (threadIdx.x == 0) atomicOr(gave_up, 1u);
        for (int it = 0; it < kWaitLimit && !landed; ++it) landed = mbar_try_wait(bar, 0);
        return;
    }
    if (!landed) landed = mbar_try_wait(bar, 0);     // returns at once; orders this thread after the copies

    SegCursor cur;
    bool have_cur = false;
    for (uint32_t e = threadIdx.x * 4u; e < cnt; e += BLK * 4u) {
        const uint64_t e0 = a.seg_base + t0 + e;
        if (!have_cur) { cur = seg_find(e0, a); have_cur = true; }
        seg_seek(cur, e0, a);
        float4 g = *reinterpret_cast<const float4*>(sg + e);
        float4 p = *reinterpret_cast<const float4*>(sp + e);
        float4 m = *reinterpret_cast<const float4*>(sm + e);
        float4 v = *reinterpret_cast<const float4*>(sv + e);
        float* pf = reinterpret_cast<float*>(&p);
        float* mf = reinterpret_cast<float*>(&m);
        float* vf = reinterpret_cast<float*>(&v);
        const float* gf = reinterpret_cast<const float*>(&g);
        SegCursor c = cur;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            seg_seek(c, e0 + q, a);
            adam_element(pf[q], mf[q], vf[q], gf[q], c.decay != 0, a);
        }
        *reinterpret_cast<float4*>(sp + e) = p;
        *reinterpret_cast<float4*>(sm + e) = m;
        *reinterpret_cast<float4*>(sv + e) = v;
        *reinterpret_cast<uint2*>(srep + e) = bf16_pack4(p);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // shared-memory writes visible to the copy engine
    __syncthreads();
    if (threadIdx.x == 0) {
        bulk_store(a.p + t0, sp, bytes);
        bulk_store(a.m + t0, sm, bytes);
        bulk_store(a.v + t0, sv, bytes);
        bulk_store(a.rep + t0, srep, cnt * 2u);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory must outlive the reads
    }
}

template <int TILE, int BLK>
cudaError_t run_adamw_bulk(const alsgd_sweep_buffers& b, uint32_t, cudaStream_t s) {
    if (b.n % 8 != 0 || !b.adam_rep) return cudaErrorInvalidValue;
    const uintptr_t all = reinterpret_cast<uintptr_t>(b.adam_p) | reinterpret_cast<uintptr_t>(b.adam_m) |
                          reinterpret_cast<uintptr_t>(b.adam_v) | reinterpret_cast<uintptr_t>(b.adam_g) |
                          reinterpret_cast<uintptr_t>(b.adam_rep);
    if (all % 16) return cudaErrorInvalidValue;
    AdamArgs a{};
    a.p = b.adam_p; a.p_src = b.adam_p; a.m = b.adam_m; a.v = b.adam_v; a.g = b.adam_g; a.rep = b.adam_rep;
    a.seg_end = b.seg_end; a.seg_decay = b.seg_decay; a.n_seg = b.n_seg;
    a.n = b.n; a.seg_base = 0;
    a.b1 = 0.9f; a.b2 = 0.95f; a.omb1 = 1.0f - a.b1; a.omb2 = 1.0f - a.b2;
    a.bc1 = 0.65f; a.bc2 = 0.4f; a.eps = 1e-8f; a.lr = 1e-3f; a.wd = 0.1f;
    auto kern = adamw_bulk_kernel<TILE, BLK>;
    constexpr int smem_bytes = TILE * 18;                   // g, p, m, v fp32 + bf16 replica
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    const uint64_t tiles = (b.n + TILE - 1) / TILE;
    if (tiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    kern<<<(unsigned)tiles, BLK, smem_bytes, s>>>(a, b.diag_flags + 7);
    return cudaGetLastError();
}

#define ADB(TILE, BLK) \
    {{ALSGD_SWEEP_ADAMW, 0, 0, TILE / (BLK * 4), BLK, 1, 0, 0, 0, TILE}, &run_adamw_bulk<TILE, BLK>},
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
    ADB(1024, 128) ADB(1024, 256) ADB(2048, 128) ADB(2048, 256) ADB(4096, 128) ADB(4096, 256) ADB(8192, 256)
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

// Device code of the sm_100a kernels of the asynchronous Local-SGD server step and the inner AdamW
// step, as templates over the launch shape.  alsgd_kernels.cu instantiates the shapes the library
// runs; alsgd_sweep.cu instantiates many shapes of the same bodies for the launch-shape benchmark.
//
// Every kernel here is a pure stream over flat fp32 vectors (0.3-0.6 flop per byte), so the design
// goal is HBM bandwidth: 128-bit coalesced accesses, several independent vectors in flight per
// thread, one pass over theta / Delta / m no matter how many workers arrive, and the re-seed of the
// dispatched workers written from registers in the same pass.  Consecutive launches walk the vectors
// in opposite directions (ArriveArgs::reverse, AdamArgs::reverse), so that the part of a worker's
// state the previous launch touched last, which the 126 MB L2 still holds, is the part the next launch
// touches first: back-to-back AdamW steps of one worker gain 1.3 % at 110M elements, 2.9 % at 59M,
// 6.4 % at 23M.  For the same reason loads and stores carry no evict-first hint (ALSGD_STREAM_HINTS
// = 0; with the hints the same kernels measured 0.5-1 % slower).
// Each block handles exactly one tile and exits (PERSIST = false): on B200 this measured 15-20 %
// faster than a persistent grid-stride loop of the same body, because the block scheduler keeps
// fresh blocks issuing loads while older ones are still storing, instead of all resident blocks
// marching through load and store phases together.
//
// Arithmetic contract: every fp32 operation is a separate IEEE-754 round-to-nearest operation in
// the order Algorithm 3 states it (compiled with -fmad=false, IEEE division and square root, no
// flush-to-zero), so results do not depend on the launch shape.  The only fused multiply-adds are the
// explicit ones of the optional diagnostics, which feed no state.  PK (the two-lane f32x2 instructions
// of sm_100) exists for the launch-shape benchmark only and is off in every shape the library runs:
// see Lanes below.
#pragma once
#include "alsgd_kernels.cuh"

#include <cuda_runtime.h>

namespace alsgd {
namespace kern {

// Which model the pseudo-gradient is taken against, and how many snapshot vectors a launch reads.
enum : int {
    kBasePerArrival = 0,  // arrival j reads its own dispatch snapshot base[j]
    kBaseShared = 1,      // all arrivals were dispatched with the same snapshot: base[0] is read once
    kBaseCurrent = 2      // the running theta: no snapshot is read
};

// Access codes recorded by the debug guard (one bit per kind of vector).
enum : unsigned {
    kGuardTheta = 1u, kGuardDelta = 2u, kGuardMom = 4u, kGuardWorkerP = 8u, kGuardBase = 16u,
    kGuardSeed = 32u, kGuardAdamP = 64u, kGuardAdamM = 128u, kGuardAdamV = 256u, kGuardReplica = 512u
};

// ---------------------------------------------------------------------------------------------
// Guarded accesses.  In the normal build the guard is empty and every access is a plain streaming
// load or store.  With ALSGD_DEBUG_BOUNDS every access to an arena-owned vector is first checked
// against the arena's byte range and its natural alignment; a violation records a code in the
// context's error word and the access is skipped (loads give zero), so a wrong slice or worker
// pointer shows up as a status from alsgd_sync instead of a memory fault.
// ---------------------------------------------------------------------------------------------
#ifdef ALSGD_DEBUG_BOUNDS
__device__ __forceinline__ bool guard_ok(const DebugGuard& g, const void* p, unsigned bytes, unsigned code) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(p);
    if (x >= g.lo && x + bytes <= g.hi && (x % bytes) == 0) return true;
    if (g.err) atomicOr(g.err, code);
    return false;
}
#define ALSGD_GUARD(g, p, bytes, code) guard_ok(g, p, bytes, code)
#else
#define ALSGD_GUARD(g, p, bytes, code) true
#endif

#ifndef ALSGD_STREAM_HINTS
#define ALSGD_STREAM_HINTS 0      // 1: ld.global.cs / st.global.cs (evict-first) on every stream
#endif
__device__ __forceinline__ float4 ld4(const DebugGuard& g, const float4* p, unsigned code) {
    if (!ALSGD_GUARD(g, p, 16, code)) return make_float4(0.f, 0.f, 0.f, 0.f);
#if ALSGD_STREAM_HINTS
    return __ldcs(p);
#else
    return *p;
#endif
}
__device__ __forceinline__ void st4(const DebugGuard& g, float4* p, float4 v, unsigned code) {
    if (!ALSGD_GUARD(g, p, 16, code)) return;
#if ALSGD_STREAM_HINTS
    __stcs(p, v);
#else
    *p = v;
#endif
}
__device__ __forceinline__ void st2(const DebugGuard& g, uint2* p, uint2 v, unsigned code) {
    if (!ALSGD_GUARD(g, p, 8, code)) return;
#if ALSGD_STREAM_HINTS
    __stcs(p, v);
#else
    *p = v;
#endif
}
__device__ __forceinline__ float ld1(const DebugGuard& g, const float* p, unsigned code) {
    if (!ALSGD_GUARD(g, p, 4, code)) return 0.f;
    return *p;
}
__device__ __forceinline__ void st1(const DebugGuard& g, float* p, float v, unsigned code) {
    if (!ALSGD_GUARD(g, p, 4, code)) return;
    *p = v;
}
__device__ __forceinline__ void st1h(const DebugGuard& g, uint16_t* p, uint16_t v, unsigned code) {
    if (!ALSGD_GUARD(g, p, 2, code)) return;
    *p = v;
}

// bf16 round-to-nearest-even on the raw bits; NaN becomes a quiet NaN with the sign kept.
__device__ __forceinline__ uint32_t bf16_bits(float x) {
    const uint32_t u = __float_as_uint(x);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return ((u >> 16) & 0x8000u) | 0x7FC0u;
    return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}

__device__ __forceinline__ uint2 bf16_pack4(const float4& x) {
    uint2 r;
    r.x = bf16_bits(x.x) | (bf16_bits(x.y) << 16);
    r.y = bf16_bits(x.z) | (bf16_bits(x.w) << 16);
    return r;
}

// ---------------------------------------------------------------------------------------------
// Two-lane fp32 arithmetic.  PK = false is a pair of scalar IEEE operations: what the library runs.
// PK = true issues the sm_100 f32x2 instructions (one instruction, two round-to-nearest lanes,
// denormals kept).  Each packed instruction alone matches the scalar pair bit for bit, but measured
// on B200 (CUDA 12.9) a packed multiply by a scalar broadcast to both lanes followed by a packed add
// or subtract comes out as ONE fused multiply-add, despite the .rn qualifiers and -fmad=false: about
// 20 % of such results differ from the two-rounding value in the last bit.  That breaks the
// one-rounding-per-operation contract (and with it the bit-exact bf16 replicas), and the gain was
// 1.3 % at best (eight arrivals with diagnostics), so PK stays a benchmark-only variant.
// ---------------------------------------------------------------------------------------------
template <bool PK>
struct Lanes {
    static __device__ __forceinline__ float2 add(float2 a, float2 b) {
        if constexpr (PK) {
            float2 r;
            asm("{ .reg .b64 ra, rb, rc; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; add.rn.f32x2 rc, ra, rb; mov.b64 {%0, %1}, rc; }"
                : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
            return r;
        } else {
            return make_float2(a.x + b.x, a.y + b.y);
        }
    }
    static __device__ __forceinline__ float2 sub(float2 a, float2 b) {
        if constexpr (PK) {
            float2 r;
            asm("{ .reg .b64 ra, rb, rc; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; sub.rn.f32x2 rc, ra, rb; mov.b64 {%0, %1}, rc; }"
                : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
            return r;
        } else {
            return make_float2(a.x - b.x, a.y - b.y);
        }
    }
    static __device__ __forceinline__ float2 mul(float2 a, float2 b) {
        if constexpr (PK) {
            float2 r;
            asm("{ .reg .b64 ra, rb, rc; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mul.rn.f32x2 rc, ra, rb; mov.b64 {%0, %1}, rc; }"
                : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
            return r;
        } else {
            return make_float2(a.x * b.x, a.y * b.y);
        }
    }
    // Explicitly fused; used by the diagnostics only.
    static __device__ __forceinline__ float2 fma(float2 a, float2 b, float2 c) {
        if constexpr (PK) {
            float2 r;
            asm("{ .reg .b64 ra, rb, rc, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mov.b64 rc, {%6, %7}; "
                "fma.rn.f32x2 rd, ra, rb, rc; mov.b64 {%0, %1}, rd; }"
                : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
            return r;
        } else {
            return make_float2(__fmaf_rn(a.x, b.x, c.x), __fmaf_rn(a.y, b.y, c.y));
        }
    }
    static __device__ __forceinline__ float2 mul(float s, float2 b) { return mul(make_float2(s, s), b); }
};

__device__ __forceinline__ bool nonfinite_bits(float x) { return (__float_as_uint(x) & 0x7F800000u) == 0x7F800000u; }

// One arrival of Algorithm 3 on two elements.  th, d, mm carry theta, Delta, momentum.
// EXT adds the Section 4 variants: delay compensation, staleness weight, buffered outer step.
// DIAG accumulates the squares of the (unmodified) pseudo-gradient entries into acc.
template <bool PK, bool DIAG, int BASE, bool EXT>
__device__ __forceinline__ void dn_step(float2& th, float2& d, float2& mm, float2 b, float2 p, bool boundary, float w,
                                        const ArriveArgs& a, float& acc) {
    using L = Lanes<PK>;
    const float2 start = (BASE == kBaseCurrent) ? th : b;
    float2 g = L::sub(start, p);                              // pseudo-gradient
    if (DIAG) acc = __fmaf_rn(g.y, g.y, __fmaf_rn(g.x, g.x, acc));   // sum of squares (at most 16 terms per thread in fp32)
    if (EXT) {
        if (a.flags & kDelayComp) {                           // g + lambda * g*g*(theta_now - theta_at_dispatch)
            const float2 drift = L::sub(th, start);
            g = L::add(g, L::mul(L::mul(a.dc_lambda, L::mul(g, g)), drift));
        }
        if (w != 1.0f) g = L::mul(w, g);
    }
    d = L::add(d, g);                                         // Delta <- Delta + g
    if (EXT && (a.flags & kBuffered)) {
        if (boundary) {                                       // Eq. 4 (or the SGD Momentum step) on the buffer mean
            const float2 mean = L::mul(a.inv_n, d);
            const float2 mn = L::add(L::mul(a.beta, mm), mean);
            const float2 u = L::add(L::mul(a.beta2, mm), L::mul(a.one_plus_beta, mean));
            th = L::sub(th, L::mul(a.eps, u));
            mm = mn;
            d = make_float2(0.f, 0.f);
        }
        return;
    }
    const float2 gn = L::mul(a.inv_n, g);                     // g / N
    if (boundary) {
        const float2 mn = L::add(L::mul(a.beta, mm), L::mul(a.inv_n, d));   // m <- beta m + Delta/N
        const float2 u = L::add(L::mul(a.cb, mn), gn);                      // (1-cN+c) beta m + g/N
        th = L::sub(th, L::mul(a.eps, u));
        mm = mn;
        d = make_float2(0.f, 0.f);
    } else {
        const float2 u = (a.flags & kCNonZero) ? L::add(L::mul(a.cn, mm), gn) : gn;   // c beta m + g/N
        th = L::sub(th, L::mul(a.eps, u));
    }
}

// Cold path of the diagnostics: which of the K arrivals have a non-finite pseudo-gradient entry at
// element e?  Only reached when the state that came out of the hot path is not finite there (a
// non-finite entry always leaves theta or Delta non-finite, see arrive_kernel), and always before
// anything is stored at e, so every input still holds its value from before the launch.
template <int K, int BASE, bool EXT>
__device__ __noinline__ uint32_t replay_nonfinite(const ArriveArgs& a, uint64_t e) {
    uint32_t bad = 0;
    const DebugGuard& gd = a.guard;
    float2 th = make_float2(ld1(gd, a.theta + e, kGuardTheta), 0.f);
    float2 d = make_float2((a.flags & kDeltaZeroIn) ? 0.f : ld1(gd, a.delta + e, kGuardDelta), 0.f);
    float2 mm = make_float2((a.flags & kReadM) ? ld1(gd, a.mom + e, kGuardMom) : 0.f, 0.f);
    float unused = 0.f;
#pragma unroll 1
    for (int j = 0; j < K; ++j) {
        const float p = ld1(gd, a.p[j] + e, kGuardWorkerP);
        const float start = (BASE == kBaseCurrent) ? th.x : ld1(gd, a.base[BASE == kBaseShared ? 0 : j] + e, kGuardBase);
        if (nonfinite_bits(start - p)) bad |= 1u << j;
        if (BASE == kBaseCurrent)          // the next arrival's pseudo-gradient is against theta after this one
            dn_step<false, false, BASE, EXT>(th, d, mm, make_float2(0.f, 0.f), make_float2(p, 0.f),
                                             (a.boundary_mask >> j) & 1u, EXT ? a.w[j] : 1.0f, a, unused);
    }
    return bad;
}

// Sum over the 32 lanes of a warp of K values per lane with K - 1 + (5 - log2 K') shuffles instead of 5 K
// (K' = K rounded up to a power of two): in each of the first log2 K' steps a lane hands half of its values to
// its partner and adds the partner's other half to the half it keeps; afterwards every lane holds one value, and
// the remaining steps are ordinary.  On return lane l with (l & (32 / K' - 1)) == 0 holds the warp's sum of value
// j = l / (32 / K').  The order of the additions is fixed, so the result is reproducible.
template <int K>
__device__ __forceinline__ float warp_sum_transposed(float (&v)[8], int lane) {
    constexpr int KP = K <= 1 ? 1 : K <= 2 ? 2 : K <= 4 ? 4 : 8;
    int m = 16;
#pragma unroll
    for (int cnt = KP; cnt > 1; cnt >>= 1, m >>= 1) {
        const bool upper = lane & m;
#pragma unroll
        for (int i = 0; i < cnt / 2; ++i) {
            const float send = upper ? v[i] : v[i + cnt / 2];
            const float keep = upper ? v[i + cnt / 2] : v[i];
            v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, m);
        }
    }
    float s = v[0];
#pragma unroll
    for (; m > 0; m >>= 1) s = s + __shfl_xor_sync(0xFFFFFFFFu, s, m);
    return s;
}

// Programmatic dependent launch: when a kernel is launched with the stream-serialization attribute its blocks
// may be placed on the SMs while the previous kernel of the stream is still draining; they then wait here, before
// their first memory access, until that kernel has completed and its writes are visible.  launch_dependents lets
// the next kernel do the same with this one.  Without the attribute both instructions do nothing.
__device__ __forceinline__ void grid_dependency_sync() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// kernel<<<grid, block, 0, s>>>(args), optionally as a programmatic dependent launch.
template <typename Args>
inline cudaError_t launch_kernel(void (*kern)(Args), unsigned grid, unsigned block, cudaStream_t s, const Args& args, bool pdl) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, args);
}

template <int K, int V, int BLK, int MINB, bool DIAG, int BASE, bool EXT, bool PERSIST, bool PK>
__global__ void __launch_bounds__(BLK, MINB) arrive_kernel(const __grid_constant__ ArriveArgs a) {
    grid_dependency_sync();
    constexpr int KK = K > 0 ? K : 1;
    constexpr int NB = (BASE == kBasePerArrival) ? KK : 1;     // snapshot vectors held in registers
    const uint64_t nvec = a.n >> 2;
    const uint64_t tile = (uint64_t)BLK * V;
    const uint32_t flags = a.flags;
    const bool read_delta = K > 0 && !(flags & kDeltaZeroIn);
    const bool write_delta = K > 0 && !(flags & kDeltaSkipStore);
    const bool read_m = K > 0 && (flags & kReadM);
    const bool write_m = K > 0 && (flags & kWriteM);
    const bool write_theta = !(EXT && (flags & kSkipThetaStore));
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    const DebugGuard& gd = a.guard;

    float acc[KK];                                             // per arrival: sum of squares of this thread's entries
#pragma unroll
    for (int j = 0; j < KK; ++j) acc[j] = 0.f;
    uint32_t bad = 0;                                          // bit j: arrival j had a non-finite entry

    float4* __restrict__ theta4 = reinterpret_cast<float4*>(a.theta);
    float4* __restrict__ delta4 = reinterpret_cast<float4*>(a.delta);
    float4* __restrict__ mom4 = reinterpret_cast<float4*>(a.mom);

    const uint64_t n_tiles = (nvec + tile - 1) / tile;
    uint64_t tile_i = (a.reverse && !PERSIST) ? n_tiles - 1 - blockIdx.x : blockIdx.x;   // one tile per block unless PERSIST
    do {
        const uint64_t t0 = tile_i * tile;
        float4 th[V], d[V], mm[V];
        float4 b[NB][V], p[KK][V];
        // ---- issue every load of the tile before the first use
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const uint64_t i = t0 + (uint64_t)v * BLK + threadIdx.x;
            const bool ok = i < nvec;
            th[v] = ok ? ld4(gd, theta4 + i, kGuardTheta) : zero4;
            d[v] = (ok && read_delta) ? ld4(gd, delta4 + i, kGuardDelta) : zero4;
            mm[v] = (ok && read_m) ? ld4(gd, mom4 + i, kGuardMom) : zero4;
#pragma unroll
            for (int j = 0; j < K; ++j)
                p[j][v] = ok ? ld4(gd, reinterpret_cast<const float4*>(a.p[j]) + i, kGuardWorkerP) : zero4;
            if (K > 0 && BASE != kBaseCurrent) {
#pragma unroll
                for (int q = 0; q < NB; ++q)
                    b[q][v] = ok ? ld4(gd, reinterpret_cast<const float4*>(a.base[q]) + i, kGuardBase) : zero4;
            }
        }
        // ---- arithmetic and stores
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const uint64_t i = t0 + (uint64_t)v * BLK + threadIdx.x;
            if (i >= nvec) continue;
            if (K > 0) {
                float2 tl = make_float2(th[v].x, th[v].y), tu = make_float2(th[v].z, th[v].w);
                float2 dl = make_float2(d[v].x, d[v].y), du = make_float2(d[v].z, d[v].w);
                float2 ml = make_float2(mm[v].x, mm[v].y), mu = make_float2(mm[v].z, mm[v].w);
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    float4 bj = zero4;
                    if (BASE != kBaseCurrent) bj = b[BASE == kBasePerArrival ? j : 0][v];
                    const bool bnd = (a.boundary_mask >> j) & 1u;
                    const float w = EXT ? a.w[j] : 1.0f;
                    dn_step<PK, DIAG, BASE, EXT>(tl, dl, ml, make_float2(bj.x, bj.y), make_float2(p[j][v].x, p[j][v].y), bnd, w, a, acc[j]);
                    dn_step<PK, DIAG, BASE, EXT>(tu, du, mu, make_float2(bj.z, bj.w), make_float2(p[j][v].z, p[j][v].w), bnd, w, a, acc[j]);
                }
                th[v] = make_float4(tl.x, tl.y, tu.x, tu.y);
                d[v] = make_float4(dl.x, dl.y, du.x, du.y);
                mm[v] = make_float4(ml.x, ml.y, mu.x, mu.y);
                if (DIAG) {
                    // A non-finite pseudo-gradient entry leaves Delta non-finite until the next boundary, where it
                    // moves into the momentum and theta; theta takes it at once unless the outer step is buffered.
                    // So finite theta and Delta after the K arrivals prove that every entry was finite, and only
                    // otherwise are the arrivals looked at one by one.
                    float z = 0.f;
                    z = __fmaf_rn(th[v].x, 0.f, z); z = __fmaf_rn(th[v].y, 0.f, z);
                    z = __fmaf_rn(th[v].z, 0.f, z); z = __fmaf_rn(th[v].w, 0.f, z);
                    z = __fmaf_rn(d[v].x, 0.f, z); z = __fmaf_rn(d[v].y, 0.f, z);
                    z = __fmaf_rn(d[v].z, 0.f, z); z = __fmaf_rn(d[v].w, 0.f, z);
                    if (!(z == 0.f)) {
#pragma unroll 1
                        for (int e = 0; e < 4; ++e) bad |= replay_nonfinite<KK, BASE, EXT>(a, (i << 2) + e);
                    }
                }
                if (write_theta) st4(gd, theta4 + i, th[v], kGuardTheta);
                if (write_delta) st4(gd, delta4 + i, d[v], kGuardDelta);
                if (write_m) st4(gd, mom4 + i, mm[v], kGuardMom);
            }
            if (a.n_seed) {
                const uint2 packed = bf16_pack4(th[v]);
#pragma unroll
                for (int s = 0; s < kMaxSeeds; ++s) {
                    if (s < (int)a.n_seed) {
                        if (a.seed_p[s]) st4(gd, reinterpret_cast<float4*>(a.seed_p[s]) + i, th[v], kGuardSeed);
                        if (a.seed_base[s]) st4(gd, reinterpret_cast<float4*>(a.seed_base[s]) + i, th[v], kGuardSeed);
                        if (a.seed_rep[s]) st2(gd, reinterpret_cast<uint2*>(a.seed_rep[s]) + i, packed, kGuardReplica);
                    }
                }
            }
        }
        tile_i += gridDim.x;
    } while (PERSIST && tile_i < n_tiles);

    // ---- up to three trailing elements when n is not a multiple of four
    const uint64_t rem0 = nvec << 2;
    if (blockIdx.x == 0 && rem0 + threadIdx.x < a.n) {
        const uint64_t i = rem0 + threadIdx.x;
        float2 th = make_float2(ld1(gd, a.theta + i, kGuardTheta), 0.f);
        if (K > 0) {
            float2 d = make_float2(read_delta ? ld1(gd, a.delta + i, kGuardDelta) : 0.f, 0.f);
            float2 mm = make_float2(read_m ? ld1(gd, a.mom + i, kGuardMom) : 0.f, 0.f);
            float pe[KK], be[KK];
#pragma unroll
            for (int j = 0; j < K; ++j) {
                pe[j] = ld1(gd, a.p[j] + i, kGuardWorkerP);
                be[j] = (BASE == kBaseCurrent) ? 0.f : ld1(gd, a.base[BASE == kBasePerArrival ? j : 0] + i, kGuardBase);
            }
#pragma unroll
            for (int j = 0; j < K; ++j)
                dn_step<false, DIAG, BASE, EXT>(th, d, mm, make_float2(be[j], 0.f), make_float2(pe[j], 0.f),
                                                (a.boundary_mask >> j) & 1u, EXT ? a.w[j] : 1.0f, a, acc[j]);
            if (DIAG && (nonfinite_bits(th.x) || nonfinite_bits(d.x))) bad |= replay_nonfinite<KK, BASE, EXT>(a, i);
            if (write_theta) st1(gd, a.theta + i, th.x, kGuardTheta);
            if (write_delta) st1(gd, a.delta + i, d.x, kGuardDelta);
            if (write_m) st1(gd, a.mom + i, mm.x, kGuardMom);
        }
        for (uint32_t s = 0; s < a.n_seed; ++s) {
            if (a.seed_p[s]) st1(gd, a.seed_p[s] + i, th.x, kGuardSeed);
            if (a.seed_base[s]) st1(gd, a.seed_base[s] + i, th.x, kGuardSeed);
            if (a.seed_rep[s]) st1h(gd, a.seed_rep[s] + i, (uint16_t)bf16_bits(th.x), kGuardReplica);
        }
    }

    // ---- optional diagnostics: one partial sum per block per arrival, added up in a fixed order by
    //      the two diag_reduce kernels (no floating-point atomics, so the norm is reproducible run to
    //      run); one flag per arrival, raised by an atomicOr only when an entry is Inf or NaN
    if (DIAG && K > 0) {
        __shared__ float warp_sum[BLK / 32][KK];
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        constexpr int KP = K <= 1 ? 1 : K <= 2 ? 2 : K <= 4 ? 4 : 8;
        float v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = j < K ? acc[j < K ? j : 0] : 0.f;
        const float s = warp_sum_transposed<K>(v, lane);
        if ((lane & (32 / KP - 1)) == 0 && lane / (32 / KP) < K) warp_sum[warp][lane / (32 / KP)] = s;
        bad = __reduce_or_sync(0xFFFFFFFFu, bad);
        if (lane == 0 && bad) {
            for (int j = 0; j < K; ++j)
                if ((bad >> j) & 1u) atomicOr(a.nonfinite + j, 1u);
        }
        __syncthreads();
        if ((int)threadIdx.x < K) {
            double s = 0.0;
            for (int w = 0; w < BLK / 32; ++w) s += (double)warp_sum[w][threadIdx.x];   // double from here on
            a.diag_partial[(uint64_t)threadIdx.x * gridDim.x + blockIdx.x] = s;   // [arrival][block]
        }
    }
}

// Fixed-order sum of the per-block partials partial[arrival][block], in one launch that follows the pass.
// Block (r, j) adds the r-th of kDiagChunks contiguous chunks of arrival j's partials; the block of an arrival
// that finishes last (a ticket counter per arrival) adds the kDiagChunks chunk sums in index order, hands out the
// arrival's norm and non-finite flag, and puts flag and counter back to zero for the next pass.  The order of
// every addition is fixed, so the same inputs give the same bits whichever block happens to be last.
constexpr int kDiagChunks = 64;
constexpr int kDiagBlock = 256;

__global__ void __launch_bounds__(kDiagBlock) diag_reduce_kernel(const double* __restrict__ partial, uint32_t n_blocks,
                                                                 double* chunk_sum, double* __restrict__ gnorm2_out,
                                                                 unsigned int* flag_acc, unsigned int* flag_out,
                                                                 unsigned int* ticket) {
    grid_dependency_sync();
    __shared__ double lane_sum[kDiagBlock];
    __shared__ bool last;
    const uint32_t r = blockIdx.x, j = blockIdx.y;
    const uint32_t per = (n_blocks + kDiagChunks - 1) / kDiagChunks;
    const uint32_t lo = min(r * per, n_blocks), hi = min(lo + per, n_blocks);
    const double* __restrict__ row = partial + (uint64_t)j * n_blocks;
    double s = 0.0;
    for (uint32_t bidx = lo + threadIdx.x; bidx < hi; bidx += kDiagBlock) s += row[bidx];
    lane_sum[threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < kDiagBlock; ++i) t += lane_sum[i];
        chunk_sum[j * kDiagChunks + r] = t;
        __threadfence();                                        // the chunk sum is visible before the ticket is taken
        last = atomicAdd(ticket + j, 1u) == (unsigned)kDiagChunks - 1u;
    }
    __syncthreads();
    if (last && threadIdx.x == 0) {
        __threadfence();
        const volatile double* cs = chunk_sum + j * kDiagChunks;   // written by other blocks: read past L1
        double t = 0.0;
        for (int q = 0; q < kDiagChunks; ++q) t += cs[q];
        gnorm2_out[j] = t;
        flag_out[j] = atomicExch(flag_acc + j, 0u) ? 1u : 0u;
        ticket[j] = 0u;
    }
}

// ---------------------------------------------------------------------------------------------
// Inner AdamW step with decoupled weight decay, fused with the bf16 cast of the new parameters.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void adam_element(float& p, float& m, float& v, float g, bool decay, const AdamArgs& a) {
    const float mi = (a.b1 * m) + (a.omb1 * g);
    const float vi = (a.b2 * v) + (a.omb2 * (g * g));
    m = mi;
    v = vi;
    const float mh = mi / a.bc1;
    const float vh = vi / a.bc2;
    const float r = mh / (sqrtf(vh) + a.eps);
    p = decay ? (p - (a.lr * (r + (a.wd * p)))) : (p - (a.lr * r));
}

struct SegCursor {
    uint32_t idx;
    uint64_t end;
    uint32_t decay;
};

__device__ __forceinline__ void seg_seek(SegCursor& c, uint64_t e, const AdamArgs& a) {
    while (e >= c.end && c.idx + 1 < a.n_seg) {
        ++c.idx;
        c.end = __ldg(a.seg_end + c.idx);
        c.decay = __ldg(a.seg_decay + c.idx);
    }
}

__device__ __forceinline__ SegCursor seg_find(uint64_t e, const AdamArgs& a) {
    uint32_t lo = 0, hi = a.n_seg - 1;            // first segment whose end is > e
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if (__ldg(a.seg_end + mid) > e) hi = mid; else lo = mid + 1;
    }
    SegCursor c;
    c.idx = lo;
    c.end = __ldg(a.seg_end + lo);
    c.decay = __ldg(a.seg_decay + lo);
    return c;
}

// bf16 -> fp32 is exact: the 16 bits are the upper half of the binary32 pattern.
__device__ __forceinline__ float4 widen_bf16x4(uint2 b) {
    return make_float4(__uint_as_float(b.x << 16), __uint_as_float(b.x & 0xFFFF0000u),
                       __uint_as_float(b.y << 16), __uint_as_float(b.y & 0xFFFF0000u));
}

template <int V, int BLK, int MINB, bool G16, bool PERSIST>
__global__ void __launch_bounds__(BLK, MINB) adamw_kernel(const __grid_constant__ AdamArgs a) {
    grid_dependency_sync();
    const uint64_t nvec = a.n >> 2;
    const uint64_t tile = (uint64_t)BLK * V;
    float4* p4 = reinterpret_cast<float4*>(a.p);
    const float4* ps4 = reinterpret_cast<const float4*>(a.p_src);
    float4* __restrict__ m4 = reinterpret_cast<float4*>(a.m);
    float4* __restrict__ v4 = reinterpret_cast<float4*>(a.v);
    const float4* __restrict__ g4 = reinterpret_cast<const float4*>(a.g);
    const uint2* __restrict__ g2 = reinterpret_cast<const uint2*>(a.g16);
    uint2* __restrict__ rep2 = reinterpret_cast<uint2*>(a.rep);
    const DebugGuard& gd = a.guard;

    SegCursor cur;
    bool have_cur = false;

    const uint64_t n_tiles = (nvec + tile - 1) / tile;
    uint64_t tile_i = (a.reverse && !PERSIST) ? n_tiles - 1 - blockIdx.x : blockIdx.x;   // one tile per block unless PERSIST
    do {
        const uint64_t t0 = tile_i * tile;
        float4 p[V], m[V], v[V], g[V];
#pragma unroll
        for (int k = 0; k < V; ++k) {
            const uint64_t i = t0 + (uint64_t)k * BLK + threadIdx.x;
            if (i < nvec) {
#if ALSGD_STREAM_HINTS
                g[k] = G16 ? widen_bf16x4(__ldcs(g2 + i)) : __ldcs(g4 + i);   // caller's memory: not arena-guarded
#else
                g[k] = G16 ? widen_bf16x4(g2[i]) : g4[i];
#endif
                p[k] = ld4(gd, ps4 + i, kGuardAdamP);
                m[k] = ld4(gd, m4 + i, kGuardAdamM);
                v[k] = ld4(gd, v4 + i, kGuardAdamV);
            }
        }
#pragma unroll
        for (int k = 0; k < V; ++k) {
            const uint64_t i = t0 + (uint64_t)k * BLK + threadIdx.x;
            if (i >= nvec) continue;
            const uint64_t e0 = a.seg_base + (i << 2);
            if (!have_cur) { cur = seg_find(e0, a); have_cur = true; }
            seg_seek(cur, e0, a);
            float* pf = reinterpret_cast<float*>(&p[k]);
            float* mf = reinterpret_cast<float*>(&m[k]);
            float* vf = reinterpret_cast<float*>(&v[k]);
            const float* gf = reinterpret_cast<const float*>(&g[k]);
            if (e0 + 4 <= cur.end) {
                const bool dec = cur.decay != 0;
#pragma unroll
                for (int e = 0; e < 4; ++e) adam_element(pf[e], mf[e], vf[e], gf[e], dec, a);
            } else {                                   // the vector straddles a segment edge
                SegCursor c = cur;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    seg_seek(c, e0 + e, a);
                    adam_element(pf[e], mf[e], vf[e], gf[e], c.decay != 0, a);
                }
            }
            st4(gd, p4 + i, p[k], kGuardAdamP);
            st4(gd, m4 + i, m[k], kGuardAdamM);
            st4(gd, v4 + i, v[k], kGuardAdamV);
            if (a.rep) st2(gd, rep2 + i, bf16_pack4(p[k]), kGuardReplica);
        }
        tile_i += gridDim.x;
        if (PERSIST) have_cur = false;                 // the next tile is far away: search again
    } while (PERSIST && tile_i < n_tiles);

    const uint64_t rem0 = nvec << 2;
    if (blockIdx.x == 0 && rem0 + threadIdx.x < a.n) {
        const uint64_t i = rem0 + threadIdx.x;
        SegCursor c = seg_find(a.seg_base + i, a);
        float p = ld1(gd, a.p_src + i, kGuardAdamP), m = ld1(gd, a.m + i, kGuardAdamM), v = ld1(gd, a.v + i, kGuardAdamV);
        const float gi = G16 ? __uint_as_float((uint32_t)a.g16[i] << 16) : a.g[i];
        adam_element(p, m, v, gi, c.decay != 0, a);
        st1(gd, a.p + i, p, kGuardAdamP);
        st1(gd, a.m + i, m, kGuardAdamM);
        st1(gd, a.v + i, v, kGuardAdamV);
        if (a.rep) st1h(gd, a.rep + i, (uint16_t)bf16_bits(p), kGuardReplica);
    }
}

// Blocks for one tile per block over n elements (block 0 also takes the up to three trailing elements).
inline cudaError_t grid_for(uint64_t n, uint64_t tile_vecs, unsigned* grid) {
    uint64_t tiles = ((n >> 2) + tile_vecs - 1) / tile_vecs;
    if (tiles < 1) tiles = 1;
    if (tiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    *grid = (unsigned)tiles;
    return cudaSuccess;
}

}  // namespace kern
}  // namespace alsgd

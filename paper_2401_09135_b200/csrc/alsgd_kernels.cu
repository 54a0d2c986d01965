// sm_100a kernels of the asynchronous Local-SGD server step and the inner AdamW step.
//
// Every kernel here is a pure stream over flat fp32 vectors (0.3-0.6 flop per byte), so the design
// goal is HBM bandwidth: 128-bit coalesced accesses, several independent vectors in flight per
// thread, touch-once cache hints, one pass over theta / Delta / m no matter how many workers
// arrive, and the re-seed of the dispatched workers written from registers in the same pass.
// Each block handles exactly one tile and exits: on B200 this measured 15-20 % faster than a
// persistent grid-stride loop of the same body (6.6-6.9 TB/s against 5.3-6.0 TB/s), because the
// block scheduler keeps fresh blocks issuing loads while older ones are still storing, instead
// of all resident blocks marching through load and store phases together.
//
// Arithmetic contract: every fp32 operation is a separate IEEE-754 round-to-nearest operation in
// the order Algorithm 3 states it (this file is compiled with -fmad=false, IEEE division and
// square root, no flush-to-zero), so results do not depend on the launch shape.  The only fused
// multiply-adds are the explicit ones of the optional diagnostics, which feed no state.
#include "alsgd_kernels.cuh"

#include <cuda_runtime.h>

namespace alsgd {

namespace {

constexpr int kBlock = 256;

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(uint2* p, uint2 v) { __stcs(p, v); }

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

// K sequential arrivals of Algorithm 3 on one element.  th, d, mm carry theta, Delta, momentum.
// EXT adds the Section 4 variants: delay compensation, staleness weight, buffered outer step.
template <int K, bool DIAG, bool CUR, bool EXT>
__device__ __forceinline__ void dn_element(float& th, float& d, float& mm, const float* b, const float* p,
                                           const ArriveArgs& a, float* acc) {
#pragma unroll
    for (int j = 0; j < K; ++j) {
        const float start = CUR ? th : b[j];
        float g = start - p[j];                       // pseudo-gradient
        if (DIAG) {                                   // two instructions per entry:
            acc[j] = __fmaf_rn(g, g, acc[j]);         //   sum of squares (at most 16 terms per thread in fp32)
            acc[K + j] = __fmaf_rn(g, 0.0f, acc[K + j]);   // stays 0 unless an entry is Inf or NaN
        }
        if (EXT) {
            if (a.flags & kDelayComp) {               // g + lambda * g*g*(theta_now - theta_at_dispatch)
                const float drift = th - start;
                g = g + ((a.dc_lambda * (g * g)) * drift);
            }
            if (a.w[j] != 1.0f) g = a.w[j] * g;
        }
        d = d + g;                                    // Delta <- Delta + g
        if (EXT && (a.flags & kBuffered)) {
            if ((a.boundary_mask >> j) & 1u) {        // Eq. 4 on the buffer mean
                const float mean = d * a.inv_n;
                const float mn = (a.beta * mm) + mean;
                const float u = (a.beta2 * mm) + (a.one_plus_beta * mean);
                th = th - (a.eps * u);
                mm = mn;
                d = 0.0f;
            }
            continue;
        }
        const float gn = g * a.inv_n;                 // g / N
        if ((a.boundary_mask >> j) & 1u) {
            const float mn = (a.beta * mm) + (d * a.inv_n);   // m <- beta m + Delta/N
            const float u = (a.cb * mn) + gn;                 // (1-cN+c) beta m + g/N
            th = th - (a.eps * u);
            mm = mn;
            d = 0.0f;
        } else {
            const float u = (a.flags & kCNonZero) ? ((a.cn * mm) + gn) : gn;   // c beta m + g/N
            th = th - (a.eps * u);
        }
    }
}

template <int K, int V, bool DIAG, bool CUR, bool EXT>
__global__ void __launch_bounds__(kBlock) arrive_kernel(const __grid_constant__ ArriveArgs a) {
    constexpr int KK = K > 0 ? K : 1;
    const uint64_t nvec = a.n >> 2;
    const uint64_t tile = (uint64_t)kBlock * V;
    const uint32_t flags = a.flags;
    const bool read_delta = K > 0 && !(flags & kDeltaZeroIn);
    const bool write_delta = K > 0 && !(flags & kDeltaSkipStore);
    const bool read_m = K > 0 && (flags & kReadM);
    const bool write_m = K > 0 && (flags & kWriteM);
    const bool write_theta = !(EXT && (flags & kSkipThetaStore));
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);

    float acc[2 * KK];                                 // [0, K): sums of squares; [K, 2K): non-finite detectors
#pragma unroll
    for (int j = 0; j < 2 * KK; ++j) acc[j] = 0.0f;

    float4* __restrict__ theta4 = reinterpret_cast<float4*>(a.theta);
    float4* __restrict__ delta4 = reinterpret_cast<float4*>(a.delta);
    float4* __restrict__ mom4 = reinterpret_cast<float4*>(a.mom);

    {
        const uint64_t t0 = (uint64_t)blockIdx.x * tile;      // one tile per block
        float4 th[V], d[V], mm[V];
        float4 b[KK][V], p[KK][V];
        // ---- issue every load of the tile before the first use
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const uint64_t i = t0 + (uint64_t)v * kBlock + threadIdx.x;
            const bool ok = i < nvec;
            th[v] = ok ? ld_stream(theta4 + i) : zero4;
            d[v] = (ok && read_delta) ? ld_stream(delta4 + i) : zero4;
            mm[v] = (ok && read_m) ? ld_stream(mom4 + i) : zero4;
#pragma unroll
            for (int j = 0; j < K; ++j) {
                p[j][v] = ok ? ld_stream(reinterpret_cast<const float4*>(a.p[j]) + i) : zero4;
                if (!CUR) b[j][v] = ok ? ld_stream(reinterpret_cast<const float4*>(a.base[j]) + i) : zero4;
            }
        }
        // ---- arithmetic and stores
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const uint64_t i = t0 + (uint64_t)v * kBlock + threadIdx.x;
            if (i >= nvec) continue;
            if (K > 0) {
                float* thf = reinterpret_cast<float*>(&th[v]);
                float* df = reinterpret_cast<float*>(&d[v]);
                float* mf = reinterpret_cast<float*>(&mm[v]);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float be[KK], pe[KK];
#pragma unroll
                    for (int j = 0; j < K; ++j) {
                        pe[j] = reinterpret_cast<const float*>(&p[j][v])[e];
                        be[j] = CUR ? 0.f : reinterpret_cast<const float*>(&b[j][v])[e];
                    }
                    dn_element<K, DIAG, CUR, EXT>(thf[e], df[e], mf[e], be, pe, a, acc);
                }
                if (write_theta) st_stream(theta4 + i, th[v]);
                if (write_delta) st_stream(delta4 + i, d[v]);
                if (write_m) st_stream(mom4 + i, mm[v]);
            }
            if (a.n_seed) {
                const uint2 packed = bf16_pack4(th[v]);
#pragma unroll
                for (int s = 0; s < kMaxSeeds; ++s) {
                    if (s < (int)a.n_seed) {
                        if (a.seed_p[s]) st_stream(reinterpret_cast<float4*>(a.seed_p[s]) + i, th[v]);
                        if (a.seed_base[s]) st_stream(reinterpret_cast<float4*>(a.seed_base[s]) + i, th[v]);
                        if (a.seed_rep[s]) st_stream(reinterpret_cast<uint2*>(a.seed_rep[s]) + i, packed);
                    }
                }
            }
        }
    }

    // ---- up to three trailing elements when n is not a multiple of four
    const uint64_t rem0 = nvec << 2;
    if (blockIdx.x == 0 && rem0 + threadIdx.x < a.n) {
        const uint64_t i = rem0 + threadIdx.x;
        float th = a.theta[i];
        if (K > 0) {
            float d = read_delta ? a.delta[i] : 0.f;
            float mm = read_m ? a.mom[i] : 0.f;
            float be[KK], pe[KK];
#pragma unroll
            for (int j = 0; j < K; ++j) {
                pe[j] = a.p[j][i];
                be[j] = CUR ? 0.f : a.base[j][i];
            }
            dn_element<K, DIAG, CUR, EXT>(th, d, mm, be, pe, a, acc);
            if (write_theta) a.theta[i] = th;
            if (write_delta) a.delta[i] = d;
            if (write_m) a.mom[i] = mm;
        }
        for (uint32_t s = 0; s < a.n_seed; ++s) {
            if (a.seed_p[s]) a.seed_p[s][i] = th;
            if (a.seed_base[s]) a.seed_base[s][i] = th;
            if (a.seed_rep[s]) a.seed_rep[s][i] = (uint16_t)bf16_bits(th);
        }
    }

    // ---- optional diagnostics: one partial sum per block per arrival, added up in a fixed order by
    //      the two diag_reduce kernels (no floating-point atomics, so the norm is reproducible run to
    //      run); one flag per arrival, raised by an atomicOr only when an entry is Inf or NaN
    if (DIAG && K > 0) {
        __shared__ float warp_sum[kBlock / 32][KK];
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        uint32_t bad = 0;
#pragma unroll
        for (int j = 0; j < K; ++j) {
            float s = acc[j];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s = s + __shfl_down_sync(0xFFFFFFFFu, s, o);
            if (lane == 0) warp_sum[warp][j] = s;
            if (!(acc[K + j] == 0.0f)) bad |= 1u << j;
        }
        bad = __reduce_or_sync(0xFFFFFFFFu, bad);
        if (lane == 0 && bad) {
            for (int j = 0; j < K; ++j)
                if ((bad >> j) & 1u) atomicOr(a.nonfinite + j, 1u);
        }
        __syncthreads();
        if ((int)threadIdx.x < K) {
            double s = 0.0;
            for (int w = 0; w < kBlock / 32; ++w) s += (double)warp_sum[w][threadIdx.x];   // double from here on
            a.diag_partial[(uint64_t)threadIdx.x * gridDim.x + blockIdx.x] = s;   // [arrival][block]
        }
    }
}

// Two-stage, fixed-order sum of the per-block partials partial[arrival][block].
// Stage 1: block (r, j) adds the r-th of kDiagChunks contiguous chunks of arrival j's partials.
constexpr int kDiagChunks = 64;

__global__ void __launch_bounds__(kBlock) diag_reduce1_kernel(const double* __restrict__ partial, uint32_t n_blocks,
                                                              double* __restrict__ chunk_sum) {
    __shared__ double lane_sum[kBlock];
    const uint32_t r = blockIdx.x, j = blockIdx.y;
    const uint32_t per = (n_blocks + kDiagChunks - 1) / kDiagChunks;
    const uint32_t lo = r * per, hi = min(lo + per, n_blocks);
    const double* __restrict__ row = partial + (uint64_t)j * n_blocks;
    double s = 0.0;
    for (uint32_t b = lo + threadIdx.x; b < hi; b += kBlock) s += row[b];
    lane_sum[threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < kBlock; ++i) t += lane_sum[i];
        chunk_sum[j * kDiagChunks + r] = t;
    }
}

// Stage 2: thread j adds arrival j's chunk sums in order.
__global__ void diag_reduce2_kernel(const double* __restrict__ chunk_sum, uint32_t K, double* __restrict__ out) {
    const uint32_t j = threadIdx.x;
    if (j < K) {
        double t = 0.0;
        for (int r = 0; r < kDiagChunks; ++r) t += chunk_sum[j * kDiagChunks + r];
        out[j] = t;
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

template <int V, bool G16>
__global__ void __launch_bounds__(kBlock) adamw_kernel(const __grid_constant__ AdamArgs a) {
    const uint64_t nvec = a.n >> 2;
    const uint64_t tile = (uint64_t)kBlock * V;
    float4* p4 = reinterpret_cast<float4*>(a.p);
    const float4* ps4 = reinterpret_cast<const float4*>(a.p_src);
    float4* __restrict__ m4 = reinterpret_cast<float4*>(a.m);
    float4* __restrict__ v4 = reinterpret_cast<float4*>(a.v);
    const float4* __restrict__ g4 = reinterpret_cast<const float4*>(a.g);
    const uint2* __restrict__ g2 = reinterpret_cast<const uint2*>(a.g16);
    uint2* __restrict__ rep2 = reinterpret_cast<uint2*>(a.rep);

    SegCursor cur;
    bool have_cur = false;

    {
        const uint64_t t0 = (uint64_t)blockIdx.x * tile;      // one tile per block
        float4 p[V], m[V], v[V], g[V];
#pragma unroll
        for (int k = 0; k < V; ++k) {
            const uint64_t i = t0 + (uint64_t)k * kBlock + threadIdx.x;
            if (i < nvec) {
                g[k] = G16 ? widen_bf16x4(__ldcs(g2 + i)) : ld_stream(g4 + i);
                p[k] = ld_stream(ps4 + i);
                m[k] = ld_stream(m4 + i);
                v[k] = ld_stream(v4 + i);
            }
        }
#pragma unroll
        for (int k = 0; k < V; ++k) {
            const uint64_t i = t0 + (uint64_t)k * kBlock + threadIdx.x;
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
            st_stream(p4 + i, p[k]);
            st_stream(m4 + i, m[k]);
            st_stream(v4 + i, v[k]);
            if (a.rep) st_stream(rep2 + i, bf16_pack4(p[k]));
        }
    }

    const uint64_t rem0 = nvec << 2;
    if (blockIdx.x == 0 && rem0 + threadIdx.x < a.n) {
        const uint64_t i = rem0 + threadIdx.x;
        SegCursor c = seg_find(a.seg_base + i, a);
        float p = a.p_src[i], m = a.m[i], v = a.v[i];
        const float gi = G16 ? __uint_as_float((uint32_t)a.g16[i] << 16) : a.g[i];
        adam_element(p, m, v, gi, c.decay != 0, a);
        a.p[i] = p;
        a.m[i] = m;
        a.v[i] = v;
        if (a.rep) a.rep[i] = (uint16_t)bf16_bits(p);
    }
}

// ---------------------------------------------------------------------------------------------
// Launch shapes: one block per tile of kBlock * V float4 vectors (block 0 also takes the up to
// three trailing elements).
// ---------------------------------------------------------------------------------------------
cudaError_t grid_for(uint64_t n, int vecs_per_thread, unsigned* grid) {
    const uint64_t tile = (uint64_t)kBlock * vecs_per_thread;
    uint64_t tiles = ((n >> 2) + tile - 1) / tile;
    if (tiles < 1) tiles = 1;
    if (tiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    *grid = (unsigned)tiles;
    return cudaSuccess;
}

// Vectors per thread, from measurement on B200 at 110M elements (GB/s, fused re-seed of all K):
// K=1: V=1 6635, V=2 6693, V=4 6735;  K=2: V=1 6612, V=2 6689;  K=4: V=1 6576, V=2 6626;  K=8: V=1 6600.
constexpr int arrive_vecs(int K) { return K <= 1 ? 4 : (K <= 4 ? 2 : 1); }

template <int K, bool DIAG, bool CUR, bool EXT>
cudaError_t launch_arrive_k(const ArriveArgs& a, const LaunchCfg& lc, cudaStream_t s) {
    constexpr int V = arrive_vecs(K);
    auto kern = arrive_kernel<K, V, DIAG, CUR, EXT>;
    unsigned grid = 1;
    cudaError_t e = grid_for(a.n, V, &grid);
    if (e != cudaSuccess) return e;
    (void)lc;
    kern<<<grid, kBlock, 0, s>>>(a);
    if (DIAG && K > 0) {
        double* chunk_sum = a.diag_partial + (uint64_t)K * grid;        // behind the K x grid partials
        diag_reduce1_kernel<<<dim3(kDiagChunks, K), kBlock, 0, s>>>(a.diag_partial, grid, chunk_sum);
        diag_reduce2_kernel<<<1, 32, 0, s>>>(chunk_sum, K, a.gnorm2);
    }
    return cudaGetLastError();
}

template <bool DIAG, bool CUR, bool EXT>
cudaError_t launch_arrive_dc(const ArriveArgs& a, const LaunchCfg& lc, cudaStream_t s) {
    switch (a.n_arr) {
        case 0: return launch_arrive_k<0, false, false, false>(a, lc, s);
        case 1: return launch_arrive_k<1, DIAG, CUR, EXT>(a, lc, s);
        case 2: return launch_arrive_k<2, DIAG, CUR, EXT>(a, lc, s);
        case 3: return launch_arrive_k<3, DIAG, CUR, EXT>(a, lc, s);
        case 4: return launch_arrive_k<4, DIAG, CUR, EXT>(a, lc, s);
        case 5: return launch_arrive_k<5, DIAG, CUR, EXT>(a, lc, s);
        case 6: return launch_arrive_k<6, DIAG, CUR, EXT>(a, lc, s);
        case 7: return launch_arrive_k<7, DIAG, CUR, EXT>(a, lc, s);
        case 8: return launch_arrive_k<8, DIAG, CUR, EXT>(a, lc, s);
        default: return cudaErrorInvalidValue;
    }
}

template <bool DIAG, bool CUR>
cudaError_t launch_arrive_e(const ArriveArgs& a, bool extended, const LaunchCfg& lc, cudaStream_t s) {
    return extended ? launch_arrive_dc<DIAG, CUR, true>(a, lc, s) : launch_arrive_dc<DIAG, CUR, false>(a, lc, s);
}

}  // namespace

uint64_t diag_partial_count(uint64_t n) {
    const uint64_t blocks = ((n >> 2) + kBlock - 1) / kBlock + 1;    // one float4 per thread gives the most blocks
    return (blocks + kDiagChunks) * kMaxArrivals;
}

cudaError_t launch_arrive(const ArriveArgs& a, bool pg_current, bool diagnostics, bool extended, const LaunchCfg& lc, cudaStream_t s) {
    if (a.n == 0) return cudaSuccess;
    if (a.n_arr > (uint32_t)kMaxArrivals || a.n_seed > (uint32_t)kMaxSeeds) return cudaErrorInvalidValue;
    if (diagnostics) return pg_current ? launch_arrive_e<true, true>(a, extended, lc, s) : launch_arrive_e<true, false>(a, extended, lc, s);
    return pg_current ? launch_arrive_e<false, true>(a, extended, lc, s) : launch_arrive_e<false, false>(a, extended, lc, s);
}

cudaError_t launch_adamw(const AdamArgs& a, const LaunchCfg& lc, cudaStream_t s) {
    if (a.n == 0) return cudaSuccess;
    constexpr int V = 2;
    unsigned grid = 1;
    cudaError_t e = grid_for(a.n, V, &grid);
    if (e != cudaSuccess) return e;
    (void)lc;
    if (a.g16) adamw_kernel<V, true><<<grid, kBlock, 0, s>>>(a);
    else adamw_kernel<V, false><<<grid, kBlock, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace alsgd

// alsgd_pg_norm_static: pseudo-gradient diagnostics for callers that must not allocate.
//
// Some hosts embed this library where device allocation is off the table: code running inside
// another framework's memory plan, between that framework's graph launches, or in a process whose
// device memory was handed out in full at start-up.  Such a caller owns its inputs and outputs but
// has nowhere to get working memory from.  This one entry point therefore keeps its working memory
// in a fixed array that is part of the library image: every GPU that loads the library sets aside
// kStaticScratchBytes for it until the process exits, and the entry point refuses vectors that
// would need more.
//
// The computation is the diagnostics half of the arrival kernel (sum of squared pseudo-gradient
// entries, non-finite flag) as a two-stage reduction with a fixed summation order, so the sum is
// reproducible run to run.
#include "../../include/alsgd.h"

#include <cuda_runtime.h>

#include <mutex>

namespace {

constexpr int kBlock = 256;
constexpr int kVecs = 4;                                   // float4 per thread
constexpr uint64_t kTileElems = (uint64_t)kBlock * kVecs * 4;   // 4096 elements per block
constexpr uint64_t kMaxTiles = ALSGD_STATIC_MAX_ELEMS / kTileElems;
constexpr size_t kFlagBytes = 256;                         // one flag word, padded
constexpr size_t kStaticScratchBytes = kFlagBytes + kMaxTiles * sizeof(double);
constexpr int kMaxDevices = 64;

// The working memory.  In host code this name is only a handle for cudaGetSymbolAddress; it is not
// a device address and must never be passed to a kernel or to cudaMemset as one.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};                    // per device ordinal, filled on first use

// Device address of the array on `device`, which must be the current device.  The first call per device is
// also what makes a lazily loading runtime place this module (the array and the two kernels) on the device.
// The cached address belongs to the device's primary context and is stale after a reset of that context.
cudaError_t scratch_address(int device, void** out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[device] = ptr;
    }
    *out = g_scratch_addr[device];
    return cudaSuccess;
}

// Stage 1: block b reduces elements [b*4096, (b+1)*4096) to one double, in a fixed order.
__global__ void __launch_bounds__(kBlock) pg_partial_kernel(const float* __restrict__ start, const float* __restrict__ p,
                                                            uint64_t n, unsigned int* flag, double* partial) {
    const uint64_t e0 = (uint64_t)blockIdx.x * kTileElems;
    double acc = 0.0;
    bool bad = false;
    const bool vec_ok = (e0 + kTileElems <= n);
    if (vec_ok) {
        const float4* s4 = reinterpret_cast<const float4*>(start + e0);
        const float4* p4 = reinterpret_cast<const float4*>(p + e0);
        float4 sv[kVecs], pv[kVecs];
#pragma unroll
        for (int v = 0; v < kVecs; ++v) {
            sv[v] = __ldcs(s4 + v * kBlock + threadIdx.x);
            pv[v] = __ldcs(p4 + v * kBlock + threadIdx.x);
        }
#pragma unroll
        for (int v = 0; v < kVecs; ++v) {
            const float g[4] = {sv[v].x - pv[v].x, sv[v].y - pv[v].y, sv[v].z - pv[v].z, sv[v].w - pv[v].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                acc += (double)g[e] * (double)g[e];
                bad |= !isfinite(g[e]);
            }
        }
    } else {                                               // the ragged last tile, element by element
        for (int v = 0; v < kVecs; ++v) {
            for (int e = 0; e < 4; ++e) {
                const uint64_t i = e0 + ((uint64_t)(v * kBlock + threadIdx.x) << 2) + e;
                if (i < n) {
                    const float g = start[i] - p[i];
                    acc += (double)g * (double)g;
                    bad |= !isfinite(g);
                }
            }
        }
    }
    __shared__ double warp_sum[kBlock / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, o);
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = acc;
    if (__any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(flag, 1u);
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < kBlock / 32; ++w) s += warp_sum[w];
        partial[blockIdx.x] = s;
    }
}

// Stage 2: one block adds the per-tile sums in index order and writes both results.
__global__ void __launch_bounds__(kBlock) pg_final_kernel(const double* partial, uint64_t tiles, const unsigned int* flag,
                                                          double* gnorm2_out, unsigned int* nonfinite_out) {
    __shared__ double lane_sum[kBlock];
    double s = 0.0;
    for (uint64_t i = threadIdx.x; i < tiles; i += kBlock) s += partial[i];
    lane_sum[threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < kBlock; ++i) t += lane_sum[i];
        *gnorm2_out = t;
        *nonfinite_out = *flag ? 1u : 0u;
    }
}

}  // namespace

extern "C" int alsgd_pg_norm_static(const float* start, const float* p, uint64_t n, int32_t device, void* stream,
                                    double* gnorm2_out, uint32_t* nonfinite_out) {
    if (!start || !p || !gnorm2_out || !nonfinite_out || n == 0) return ALSGD_E_ARG;
    if (device < 0 || device >= kMaxDevices) return ALSGD_E_RANGE;
    if (n > ALSGD_STATIC_MAX_ELEMS) return ALSGD_E_NOMEM;       // would not fit the fixed working memory
    if ((reinterpret_cast<uintptr_t>(start) | reinterpret_cast<uintptr_t>(p)) % 16) return ALSGD_E_ARG;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return ALSGD_E_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return ALSGD_E_CUDA;
    int rc = ALSGD_OK;
    void* base = nullptr;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (scratch_address(device, &base) != cudaSuccess) rc = ALSGD_E_CUDA;
    if (rc == ALSGD_OK) {
        unsigned int* flag = static_cast<unsigned int*>(base);
        double* partial = reinterpret_cast<double*>(static_cast<unsigned char*>(base) + kFlagBytes);
        const uint64_t tiles = (n + kTileElems - 1) / kTileElems;
        // The array keeps whatever the previous call left: the flag is OR-ed into, so it starts at zero;
        // the per-tile sums are overwritten for every tile in use.
        if (cudaMemsetAsync(flag, 0, sizeof(unsigned int), s) != cudaSuccess) rc = ALSGD_E_CUDA;
        if (rc == ALSGD_OK) {
            pg_partial_kernel<<<(unsigned)tiles, kBlock, 0, s>>>(start, p, n, flag, partial);
            pg_final_kernel<<<1, kBlock, 0, s>>>(partial, tiles, flag, gnorm2_out, nonfinite_out);
            if (cudaGetLastError() != cudaSuccess) rc = ALSGD_E_CUDA;
        }
    }
    if (prev != device) cudaSetDevice(prev);
    return rc;
}

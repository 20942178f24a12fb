// ah_distances_static: squared distances ||x_i - c||^2 without a handle and
// without allocating anything.
//
// Some callers cannot allocate device memory at the moment they need these
// distances: a monitoring hook that runs inside a training job whose framework
// allocator has already claimed all of the GPU; code on a latency-critical path,
// where cudaMalloc's device-wide synchronisation would stall every other stream; a
// component that is handed raw x and c pointers and owns no ah_ctx (creating one
// allocates a workspace).  For them the per-tile partial sums that the handle-based
// path keeps in its workspace live here in a fixed array inside the library image.
//
// The array is part of every CUDA context that loads the library (2 MiB per GPU,
// held until the process exits), which is why its size is modest and fixed:
// K * (tiles rounded up to a power of two) <= AH_STATIC_SCRATCH_ENTRIES, a tile
// being 1024 parameters.  Larger problems are refused with AH_ERR_TOO_LARGE.
//
// All calls share the one array.  Nothing in it needs clearing: every entry that
// is read in a call has been written earlier in that call, and tiles that do not
// exist are treated as +0 by index, never read.  Two calls whose kernels overlap on
// the GPU (different streams, different threads) would race on it: the caller
// serialises them.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "adahess.h"

namespace {

constexpr int kTileNA = 1024;          // parameters per tile: 256 threads x float4
constexpr int kThreadsNA = 256;
constexpr int kMaxDevices = 64;

// Two rows of scratch: tile partials, and the ping-pong buffer of the reduction.
static __device__ __align__(256) double g_static_scratch[2 * AH_STATIC_SCRATCH_ENTRIES];

// In host code g_static_scratch is only a handle for the runtime, not an address a
// kernel could use; the device address is looked up once per device.
std::mutex g_setup_mutex;
double *g_scratch_dev[kMaxDevices] = {};

__device__ __forceinline__ double sq_dist4(float4 x, float4 c, int nv)
{
    const double d0 = nv > 0 ? (double)__fsub_rn(x.x, c.x) : 0.0;
    const double d1 = nv > 1 ? (double)__fsub_rn(x.y, c.y) : 0.0;
    const double d2 = nv > 2 ? (double)__fsub_rn(x.z, c.z) : 0.0;
    const double d3 = nv > 3 ? (double)__fsub_rn(x.w, c.w) : 0.0;
    return __dadd_rn(__dadd_rn(__dmul_rn(d0, d0), __dmul_rn(d1, d1)),
                     __dadd_rn(__dmul_rn(d2, d2), __dmul_rn(d3, d3)));
}

// Per tile and worker: pairwise-tree sum of (x - c)^2 over 1024 consecutive
// parameters (4 per thread, 32 lanes by butterfly, 8 warps through shared memory).
__global__ void __launch_bounds__(kThreadsNA)
tile_distance_kernel(const float *__restrict__ x, uint64_t ldx, const float *__restrict__ c,
                     uint32_t P, uint32_t ntiles_pad, double *partials)
{
    __shared__ double red[kThreadsNA / 32];
    const uint32_t tile = blockIdx.x, i = blockIdx.y;
    const uint32_t j = tile * (uint32_t)kTileNA + 4u * threadIdx.x;
    double s = 0.0;
    if (j < P) {
        const int nv = P - j >= 4u ? 4 : (int)(P - j);
        const float4 xv = *reinterpret_cast<const float4 *>(x + (uint64_t)i * ldx + j);
        const float4 cv = *reinterpret_cast<const float4 *>(c + j);
        s = sq_dist4(xv, cv, nv);
    }
#pragma unroll
    for (int off = 1; off < 32; off <<= 1)
        s = __dadd_rn(s, __shfl_xor_sync(0xffffffffu, s, off));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t[kThreadsNA / 32];
#pragma unroll
        for (int q = 0; q < kThreadsNA / 32; ++q) t[q] = red[q];
#pragma unroll
        for (int len = kThreadsNA / 32; len > 1; len >>= 1)
#pragma unroll
            for (int q = 0; q < len / 2; ++q) t[q] = __dadd_rn(t[2 * q], t[2 * q + 1]);
        partials[(uint64_t)i * ntiles_pad + tile] = t[0];
    }
}

// Upper levels of the same tree, one CTA per worker, ping-ponging between the two
// scratch rows; tile indices >= ntiles count as +0 and are never read.
__global__ void __launch_bounds__(1024)
tree_finish_kernel(double *partials, double *pong, uint32_t ntiles, uint32_t ntiles_pad,
                   double *norm2)
{
    const int i = blockIdx.x;
    double *a = partials + (uint64_t)i * ntiles_pad;
    double *b = pong + (uint64_t)i * ntiles_pad;
    uint32_t live = ntiles;
    for (uint32_t n = ntiles_pad; n > 1; n >>= 1) {
        const uint32_t half = n >> 1;
        for (uint32_t k = threadIdx.x; k < half; k += blockDim.x) {
            const double l = 2 * k < live ? a[2 * k] : 0.0;
            const double r = 2 * k + 1 < live ? a[2 * k + 1] : 0.0;
            b[k] = __dadd_rn(l, r);
        }
        __syncthreads();
        double *t = a; a = b; b = t;
        live = half;
    }
    if (threadIdx.x == 0) norm2[i] = a[0];
}

// Device address of the static scratch on the current device; looked up on the
// first call for that device.
int scratch_for_current_device(double **out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return AH_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return AH_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_dev[dev]) {
        double *ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress((void **)&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) return AH_ERR_CUDA;
        g_scratch_dev[dev] = ptr;
    }
    *out = g_scratch_dev[dev];
    return AH_OK;
}

}  // namespace

extern "C" int ah_distances_static(const float *x, uint64_t ldx, const float *c, int K, uint64_t P,
                                   double *norm2, void *cuda_stream)
{
    if (!x || !c || !norm2 || K < 1 || K > AH_MAX_WORKERS || P < 1 || P >= (1ull << 31) || ldx < P)
        return AH_ERR_INVALID_ARG;
    if ((ldx & 3u) != 0 || ((uintptr_t)x & 15u) != 0 || ((uintptr_t)c & 15u) != 0 ||
        ((uintptr_t)norm2 & 7u) != 0)
        return AH_ERR_ALIGN;
    const uint32_t ntiles = (uint32_t)((P + kTileNA - 1) / kTileNA);
    uint32_t ntiles_pad = 1;
    while (ntiles_pad < ntiles) ntiles_pad <<= 1;
    if ((uint64_t)K * ntiles_pad > (uint64_t)AH_STATIC_SCRATCH_ENTRIES) return AH_ERR_TOO_LARGE;

    double *scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != AH_OK) return rc;
    double *partials = scratch, *pong = scratch + AH_STATIC_SCRATCH_ENTRIES;

    cudaStream_t s = (cudaStream_t)cuda_stream;
    tile_distance_kernel<<<dim3(ntiles, (unsigned)K), kThreadsNA, 0, s>>>(x, ldx, c, (uint32_t)P,
                                                                        ntiles_pad, partials);
    if (cudaGetLastError() != cudaSuccess) return AH_ERR_CUDA;
    tree_finish_kernel<<<K, 1024, 0, s>>>(partials, pong, ntiles, ntiles_pad, norm2);
    if (cudaGetLastError() != cudaSuccess) return AH_ERR_CUDA;
    return AH_OK;
}

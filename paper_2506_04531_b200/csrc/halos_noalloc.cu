// halos_push_noalloc: the push step (Delta = theta - anchor, plus the squared norm of Delta) for
// callers that must not allocate.
//
// The regular path (halos_lps_push on a context created with HALOS_FLAG_STATS) reduces the squared
// norm through a per-chunk array of partial sums that the context allocates at creation.  Some
// callers cannot allocate at all: code running while a memory pool is frozen or exhausted, inside
// a latency-critical section where an allocator call may block or synchronise the device, or in a
// host process whose policy forbids cudaMalloc after start-up.  For them the partial sums live in a
// fixed file-scope device array below.  Its price: kMaxChunks * 8 bytes = 512 KB of device memory on
// every GPU that loads this library, held until the process exits, and a hard size limit.
//
// The array is shared by every call.  Each call overwrites exactly the partials it reads back
// (slots [0, number of chunks)), so nothing has to start at zero and stale contents from an earlier,
// larger call are never read.  Two calls whose kernels overlap on the GPU (different streams, or
// different host threads on different streams) race on the array: serialise them.
#include "halos.h"

#include <cuda_runtime.h>
#include <mutex>
#include <stdint.h>

constexpr uint32_t kChunkElems = 8192;
constexpr uint32_t kMaxChunks = (uint32_t)(HALOS_NOALLOC_MAX_ELEMS / kChunkElems);  // 65536
static_assert((unsigned long long)kMaxChunks * kChunkElems == HALOS_NOALLOC_MAX_ELEMS, "limit must be whole chunks");
constexpr int kMaxDevices = 64;

// The scratch.  In host code this name is only a handle for cudaGetSymbolAddress; the device
// address it yields is what kernels receive.
static __device__ __align__(256) double g_partials[kMaxChunks];

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float4 ld_stream(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void st_stream(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

// Sum over the CTA in a fixed order (shuffle tree per warp, then warp sums in order); valid in thread 0.
__device__ __forceinline__ double block_sum(double v, double* smem /* kThreads / 32 doubles */) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) smem[threadIdx.x >> 5] = v;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) total += smem[w];
    }
    return total;
}

std::mutex g_mu;
double* g_partials_addr[kMaxDevices] = {nullptr};  // per device, filled on the first call there

// Delta for one chunk of a flat vector and the chunk's sum of squares into partials[blockIdx.x].
__global__ void __launch_bounds__(kThreads)
push_flat_kernel(const float* __restrict__ th, const float* __restrict__ an, float* __restrict__ ob,
                 unsigned long long n, double* __restrict__ partials, int vec_ok) {
    const unsigned long long begin = (unsigned long long)blockIdx.x * kChunkElems;
    const uint32_t count = (uint32_t)((n - begin) < kChunkElems ? (n - begin) : kChunkElems);
    th += begin;
    an += begin;
    ob += begin;
    float acc = 0.f;
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = count >> 2;
        for (uint32_t base = 0; base < nvec; base += kThreads * 4) {
            float4 vx[4], va[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    vx[u] = ld_stream(th + 4ull * v);
                    va[u] = ld_stream(an + 4ull * v);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    float4 D;
                    D.x = __fsub_rn(vx[u].x, va[u].x);
                    D.y = __fsub_rn(vx[u].y, va[u].y);
                    D.z = __fsub_rn(vx[u].z, va[u].z);
                    D.w = __fsub_rn(vx[u].w, va[u].w);
                    st_stream(ob + 4ull * v, D);
                    acc = fmaf(D.x, D.x, fmaf(D.y, D.y, fmaf(D.z, D.z, fmaf(D.w, D.w, acc))));
                }
            }
        }
        done = nvec << 2;
    }
    for (uint32_t j = done + threadIdx.x; j < count; j += kThreads) {
        const float D = __fsub_rn(th[j], an[j]);
        ob[j] = D;
        acc = fmaf(D, D, acc);
    }
    __shared__ double red[kThreads / 32];
    const double t = block_sum((double)acc, red);
    if (threadIdx.x == 0) partials[blockIdx.x] = t;
}

// One CTA adds partials[0, n_chunks) in a fixed order and writes the total.
__global__ void __launch_bounds__(kThreads)
sum_partials_kernel(const double* __restrict__ partials, uint32_t n_chunks, double* __restrict__ out) {
    double v = 0.0;
    for (uint32_t c = threadIdx.x; c < n_chunks; c += kThreads) v += partials[c];
    __shared__ double red[kThreads / 32];
    const double t = block_sum(v, red);
    if (threadIdx.x == 0) *out = t;
}

}  // namespace

extern "C" int halos_push_noalloc(int32_t device, void* stream, const float* theta_dev, const float* anchor_dev,
                                  float* Delta_dev, uint64_t n, double* sqnorm_dev) {
    if (n > HALOS_NOALLOC_MAX_ELEMS) return HALOS_ERR_UNSUPPORTED;  // before anything is touched
    if (device < 0 || device >= kMaxDevices) return HALOS_ERR_INVALID_ARG;
    if (!sqnorm_dev || (n && (!theta_dev || !anchor_dev || !Delta_dev))) return HALOS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(theta_dev) | reinterpret_cast<uintptr_t>(anchor_dev) |
         reinterpret_cast<uintptr_t>(Delta_dev)) & 3)
        return HALOS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(sqnorm_dev) & 7) return HALOS_ERR_INVALID_ARG;  // a double is stored through it
    if (cudaSetDevice(device) != cudaSuccess) {
        (void)cudaGetLastError();
        return HALOS_ERR_CUDA;
    }
    double* partials = nullptr;
    {
        // Set-up, once per device, with that device current: ask the runtime where this device's
        // copy of the scratch array lives.
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_partials_addr[device]) {
            double* p = nullptr;
            if (cudaGetSymbolAddress((void**)&p, g_partials) != cudaSuccess || !p) {
                (void)cudaGetLastError();
                return HALOS_ERR_CUDA;
            }
            // Load both kernels (and with them the module that holds the scratch array) now, so that
            // this first call is the only one that can make the runtime take device memory.
            cudaFuncAttributes fa;
            if (cudaFuncGetAttributes(&fa, push_flat_kernel) != cudaSuccess ||
                cudaFuncGetAttributes(&fa, sum_partials_kernel) != cudaSuccess) {
                (void)cudaGetLastError();
                return HALOS_ERR_CUDA;
            }
            g_partials_addr[device] = p;
        }
        partials = g_partials_addr[device];
    }
    cudaStream_t st = (cudaStream_t)stream;
    const uint32_t n_chunks = (uint32_t)((n + kChunkElems - 1) / kChunkElems);
    if (n_chunks) {
        const int vec_ok = ((reinterpret_cast<uintptr_t>(theta_dev) | reinterpret_cast<uintptr_t>(anchor_dev) |
                             reinterpret_cast<uintptr_t>(Delta_dev)) & 15) == 0;
        push_flat_kernel<<<n_chunks, kThreads, 0, st>>>(theta_dev, anchor_dev, Delta_dev, (unsigned long long)n,
                                                        partials, vec_ok);
    }
    sum_partials_kernel<<<1, kThreads, 0, st>>>(partials, n_chunks, sqnorm_dev);
    if (cudaGetLastError() != cudaSuccess) return HALOS_ERR_CUDA;
    return HALOS_OK;
}

// CUDA twin of the synthetic input generator (harness only; not part of the update path and not
// linked into the HALoS library).  out[j] = cast( base + sigma_k * z(key, lo + j) ) where base is
// either a per-tensor constant (model initialisation) or the worker's start snapshot (stand-in for
// H local training steps), k is the tensor that global index lo + j falls in, and z is the
// Irwin-Hall(8) unit noise of the counter-based generator described in inputs/gen.py.  Integer
// steps are exact and each floating-point step is a separately rounded fp32 operation, so the
// result equals the numpy generator bit for bit.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ull;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z;
}

__device__ __forceinline__ int lane_sum(unsigned long long h) {
    return (int)(h & 0xFFFF) + (int)((h >> 16) & 0xFFFF) + (int)((h >> 32) & 0xFFFF) + (int)(h >> 48);
}

__device__ __forceinline__ float unit_noise(unsigned long long key, unsigned long long idx) {
    const unsigned long long x = key + idx * 0x9E3779B97F4A7C15ull;
    const int s = lane_sum(mix64(x)) + lane_sum(mix64(x ^ 0xD1B54A32D192ED03ull));
    return __fmul_rn((float)(s - 262140), 0x1.3988e2p-16f);
}

// dtype: 0 = fp32, 1 = bf16 (16-bit patterns)
__global__ void synth_kernel(void* out, const void* in, int dtype, const float* __restrict__ base_tbl,
                             const float* __restrict__ sigma_tbl, const unsigned long long* __restrict__ tensor_off,
                             uint32_t n_tensors, unsigned long long key, unsigned long long lo, unsigned long long n) {
    unsigned long long j = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    for (; j < n; j += stride) {
        const unsigned long long g = lo + j;
        uint32_t a = 0, b = n_tensors;  // largest k with tensor_off[k] <= g
        while (b - a > 1) {
            const uint32_t mid = (a + b) >> 1;
            if (tensor_off[mid] <= g) a = mid; else b = mid;
        }
        const float z = unit_noise(key, g);
        float base;
        if (in) {
            base = dtype == 0 ? ((const float*)in)[j]
                              : __uint_as_float((uint32_t)((const uint16_t*)in)[j] << 16);
        } else {
            base = base_tbl[a];
        }
        const float v = __fadd_rn(base, __fmul_rn(sigma_tbl[a], z));
        if (dtype == 0) ((float*)out)[j] = v;
        else ((uint16_t*)out)[j] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
    }
}

}  // namespace

extern "C" {

// All pointers are device pointers; out/in cover global indices [lo, lo+n).  in may be NULL (then
// base_tbl is used).  Returns the cudaError_t of the launch.
int halos_synth_fill(void* out, const void* in, int dtype, const float* base_tbl, const float* sigma_tbl,
                     const unsigned long long* tensor_off, uint32_t n_tensors, unsigned long long key,
                     unsigned long long lo, unsigned long long n, void* stream) {
    if (n == 0) return 0;
    unsigned long long blocks = (n + 255) / 256;
    if (blocks > 148ull * 16) blocks = 148ull * 16;
    synth_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(out, in, dtype, base_tbl, sigma_tbl, tensor_off,
                                                                      n_tensors, key, lo, n);
    return (int)cudaGetLastError();
}

}  // extern "C"

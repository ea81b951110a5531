// Fused, bandwidth-bound update kernels of the HALoS server path for sm_100a.
//
// One launch walks every tensor of the model through a chunk table built at context creation
// (the multi-tensor chunk scheduler): chunk c = {begin, count, tensor} is a run of `count`
// consecutive elements of the packed state starting at global element `begin`, never crossing a
// tensor boundary.  One CTA processes one chunk.  Inside a chunk every thread moves 128-bit
// vectors; all loads of an unrolled batch are issued before the first use so that each SM keeps
// several tens of KB in flight.  Every buffer is read once and written once per event; the
// displacement delta, the momentum update, the model update, the worker's new start snapshot and
// (when due) Delta are formed in registers in the same pass.
//
// Rounding discipline (mirrors the definition, one rounding per written operation):
//   d  = h - s                      __fsub_rn
//   m' = beta m + d                 __fmaf_rn
//   u  = beta m' + ((1-beta) d)     __fmul_rn then __fmaf_rn
//   x' = eta u + x                  __fmaf_rn
//   merge: x' = alpha y + ((1-alpha) x)
// No fast-math, no implicit contraction (explicit intrinsics are immune to -fmad).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace halos {

struct Chunk {
    unsigned long long begin;  // global element index of the first element
    uint32_t count;            // elements in this chunk
    uint32_t tensor;           // tensor the chunk belongs to
};

// Compile-time tuning knobs (the defaults are the measured best on B200; see profiles/).
#ifndef HALOS_THREADS
#define HALOS_THREADS 256
#endif
#ifndef HALOS_UNROLL
#define HALOS_UNROLL 4
#endif
#ifndef HALOS_STREAM_HINT
#define HALOS_STREAM_HINT 1
#endif
constexpr int kThreads = HALOS_THREADS;

// ---------------------------------------------------------------- element helpers
__device__ __forceinline__ void model_update(float& x, float& m, float d, float eta, float beta, float omb) {
    float m1 = __fmaf_rn(beta, m, d);
    float u = __fmaf_rn(beta, m1, __fmul_rn(omb, d));
    x = __fmaf_rn(eta, u, x);
    m = m1;
}
__device__ __forceinline__ float merge(float x, float y, float alpha, float oma) {
    return __fmaf_rn(alpha, y, __fmul_rn(oma, x));
}
__device__ __forceinline__ float bf16_widen(uint32_t h16) { return __uint_as_float(h16 << 16); }
__device__ __forceinline__ uint32_t bf16_narrow(float x) {
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x));  // round to nearest even
}

// ---------------------------------------------------------------- 128-bit streaming access
// State is touched once per event and the working set is far larger than L2: evict-first hints.
template <bool STREAM>
__device__ __forceinline__ float4 ld4(const float* p) {
    return STREAM ? __ldcs(reinterpret_cast<const float4*>(p)) : *reinterpret_cast<const float4*>(p);
}
template <bool STREAM>
__device__ __forceinline__ void st4(float* p, float4 v) {
    if (STREAM) __stcs(reinterpret_cast<float4*>(p), v);
    else *reinterpret_cast<float4*>(p) = v;
}
template <bool STREAM>
__device__ __forceinline__ uint2 ld4h(const uint16_t* p) {  // four bf16
    return STREAM ? __ldcs(reinterpret_cast<const uint2*>(p)) : *reinterpret_cast<const uint2*>(p);
}
template <bool STREAM>
__device__ __forceinline__ void st4h(uint16_t* p, uint2 v) {
    if (STREAM) __stcs(reinterpret_cast<uint2*>(p), v);
    else *reinterpret_cast<uint2*>(p) = v;
}
__device__ __forceinline__ float4 widen4(uint2 v) {
    return make_float4(bf16_widen(v.x & 0xffffu), bf16_widen(v.x >> 16), bf16_widen(v.y & 0xffffu),
                       bf16_widen(v.y >> 16));
}
__device__ __forceinline__ uint2 narrow4(float4 v) {
    return make_uint2(bf16_narrow(v.x) | (bf16_narrow(v.y) << 16), bf16_narrow(v.z) | (bf16_narrow(v.w) << 16));
}

// worker-dtype traits: W = float (fp32 copies) or uint16_t (bf16 copies)
template <class W> struct WTraits;
template <> struct WTraits<float> {
    template <bool S> static __device__ __forceinline__ float4 load4(const float* p) { return ld4<S>(p); }
    template <bool S> static __device__ __forceinline__ void store4(float* p, float4 v) { st4<S>(p, v); }
    static __device__ __forceinline__ float load1(const float* p) { return *p; }
    static __device__ __forceinline__ void store1(float* p, float v) { *p = v; }
    static constexpr uintptr_t kVecAlignMask = 15;
};
template <> struct WTraits<uint16_t> {
    template <bool S> static __device__ __forceinline__ float4 load4(const uint16_t* p) { return widen4(ld4h<S>(p)); }
    template <bool S> static __device__ __forceinline__ void store4(uint16_t* p, float4 v) { st4h<S>(p, narrow4(v)); }
    static __device__ __forceinline__ float load1(const uint16_t* p) { return bf16_widen(*p); }
    static __device__ __forceinline__ void store1(uint16_t* p, float v) { *p = (uint16_t)bf16_narrow(v); }
    static constexpr uintptr_t kVecAlignMask = 7;
};

// ---------------------------------------------------------------- block reduction (statistics only)
// Deterministic: fixed shuffle tree inside a warp, then warp 0 adds the warp sums in order.
__device__ __forceinline__ double block_sum(double v, double* smem /* kThreads/32 doubles */) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) total += smem[w];
    }
    return total;  // valid in thread 0
}

// =====================================================================================================
// ARRIVE: delta + LPS ModelUpdate + schedule copy (+ Delta when PUSH)        Alg. 1 lines 25, 10-14
// =====================================================================================================
template <class W>
struct ArriveArgs {
    const W* h_flat;            // worker result theta_{t,H}: flat ...
    const W* const* h_ptrs;     // ... or per-tensor pointer table (device array)
    const unsigned long long* tensor_off;  // [n_tensors+1] global element offset of each tensor
    W* th0;                     // worker start snapshot theta_{t,0}  (read, then rewritten with theta_t)
    float* th;                  // LPS model
    float* ml;                  // LPS momentum
    const float* anchor;        // theta_{t_last}      (PUSH only)
    float* outbox;              // Delta               (PUSH only)
    double* partial_delta;      // [n_chunks] sum delta^2 per chunk (STATS only)
    double* partial_Delta;      // [n_chunks] sum Delta^2 per chunk (STATS && PUSH)
    float eta, beta, omb;
};

template <class W, bool PUSH, bool STATS, int UNROLL, bool STREAM>
__global__ void __launch_bounds__(kThreads)
arrive_kernel(const Chunk* __restrict__ chunks, ArriveArgs<W> a) {
    using T = WTraits<W>;
    const Chunk c = chunks[blockIdx.x];
    const W* h = a.h_flat ? a.h_flat + c.begin : a.h_ptrs[c.tensor] + (c.begin - a.tensor_off[c.tensor]);
    W* s0 = a.th0 + c.begin;
    float* th = a.th + c.begin;
    float* ml = a.ml + c.begin;
    const float* an = PUSH ? a.anchor + c.begin : nullptr;
    float* ob = PUSH ? a.outbox + c.begin : nullptr;
    const float eta = a.eta, beta = a.beta, omb = a.omb;
    float acc_d = 0.f, acc_D = 0.f;

    const bool vec_ok = ((c.begin & 3ull) == 0) && ((reinterpret_cast<uintptr_t>(h) & T::kVecAlignMask) == 0);
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count >> 2;
        for (uint32_t base = 0; base < nvec; base += kThreads * UNROLL) {
            float4 vh[UNROLL], vs[UNROLL], vx[UNROLL], vm[UNROLL], va[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    vh[u] = T::template load4<STREAM>(h + 4ull * v);
                    vs[u] = T::template load4<STREAM>(s0 + 4ull * v);
                    vx[u] = ld4<STREAM>(th + 4ull * v);
                    vm[u] = ld4<STREAM>(ml + 4ull * v);
                    if (PUSH) va[u] = ld4<STREAM>(an + 4ull * v);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    float4 d;
                    d.x = __fsub_rn(vh[u].x, vs[u].x);
                    d.y = __fsub_rn(vh[u].y, vs[u].y);
                    d.z = __fsub_rn(vh[u].z, vs[u].z);
                    d.w = __fsub_rn(vh[u].w, vs[u].w);
                    model_update(vx[u].x, vm[u].x, d.x, eta, beta, omb);
                    model_update(vx[u].y, vm[u].y, d.y, eta, beta, omb);
                    model_update(vx[u].z, vm[u].z, d.z, eta, beta, omb);
                    model_update(vx[u].w, vm[u].w, d.w, eta, beta, omb);
                    st4<STREAM>(th + 4ull * v, vx[u]);
                    st4<STREAM>(ml + 4ull * v, vm[u]);
                    T::template store4<STREAM>(s0 + 4ull * v, vx[u]);
                    if (STATS) acc_d = fmaf(d.x, d.x, fmaf(d.y, d.y, fmaf(d.z, d.z, fmaf(d.w, d.w, acc_d))));
                    if (PUSH) {
                        float4 D;
                        D.x = __fsub_rn(vx[u].x, va[u].x);
                        D.y = __fsub_rn(vx[u].y, va[u].y);
                        D.z = __fsub_rn(vx[u].z, va[u].z);
                        D.w = __fsub_rn(vx[u].w, va[u].w);
                        st4<STREAM>(ob + 4ull * v, D);
                        if (STATS) acc_D = fmaf(D.x, D.x, fmaf(D.y, D.y, fmaf(D.z, D.z, fmaf(D.w, D.w, acc_D))));
                    }
                }
            }
        }
        done = nvec << 2;
    }
    // ragged tail (or a whole chunk whose pointers do not share 16-byte alignment): scalar
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads) {
        float d = __fsub_rn(T::load1(h + j), T::load1(s0 + j));
        float x = th[j], m = ml[j];
        model_update(x, m, d, eta, beta, omb);
        th[j] = x;
        ml[j] = m;
        T::store1(s0 + j, x);
        if (STATS) acc_d = fmaf(d, d, acc_d);
        if (PUSH) {
            float D = __fsub_rn(x, an[j]);
            ob[j] = D;
            if (STATS) acc_D = fmaf(D, D, acc_D);
        }
    }
    if (STATS) {
        __shared__ double red[kThreads / 32];
        double t = block_sum((double)acc_d, red);
        if (threadIdx.x == 0) a.partial_delta[blockIdx.x] = t;
        if (PUSH) {
            __syncthreads();
            double t2 = block_sum((double)acc_D, red);
            if (threadIdx.x == 0) a.partial_Delta[blockIdx.x] = t2;
        }
    }
}

// =====================================================================================================
// PUSH alone: Delta = theta_t - theta_{t_last}                                   Alg. 1 line 14
// =====================================================================================================
struct PushArgs {
    const float* th;
    const float* anchor;
    float* outbox;
    double* partial_Delta;
};

template <bool STATS, int UNROLL, bool STREAM>
__global__ void __launch_bounds__(kThreads)
push_kernel(const Chunk* __restrict__ chunks, PushArgs a) {
    const Chunk c = chunks[blockIdx.x];
    const float* th = a.th + c.begin;
    const float* an = a.anchor + c.begin;
    float* ob = a.outbox + c.begin;
    float acc = 0.f;
    uint32_t done = 0;
    if ((c.begin & 3ull) == 0) {
        const uint32_t nvec = c.count >> 2;
        for (uint32_t base = 0; base < nvec; base += kThreads * UNROLL) {
            float4 vx[UNROLL], va[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    vx[u] = ld4<STREAM>(th + 4ull * v);
                    va[u] = ld4<STREAM>(an + 4ull * v);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    float4 D;
                    D.x = __fsub_rn(vx[u].x, va[u].x);
                    D.y = __fsub_rn(vx[u].y, va[u].y);
                    D.z = __fsub_rn(vx[u].z, va[u].z);
                    D.w = __fsub_rn(vx[u].w, va[u].w);
                    st4<STREAM>(ob + 4ull * v, D);
                    if (STATS) acc = fmaf(D.x, D.x, fmaf(D.y, D.y, fmaf(D.z, D.z, fmaf(D.w, D.w, acc))));
                }
            }
        }
        done = nvec << 2;
    }
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads) {
        float D = __fsub_rn(th[j], an[j]);
        ob[j] = D;
        if (STATS) acc = fmaf(D, D, acc);
    }
    if (STATS) {
        __shared__ double red[kThreads / 32];
        double t = block_sum((double)acc, red);
        if (threadIdx.x == 0) a.partial_Delta[blockIdx.x] = t;
    }
}

// =====================================================================================================
// GPS: global ModelUpdate + snapshot of Theta_i into the sender's inbox          Alg. 1 lines 2-4
// =====================================================================================================
struct GpsArgs {
    const float* outbox;  // Delta received
    float* Theta;
    float* Mg;
    float* inbox;         // Theta_i sent back
    float eta, beta, omb;
};

template <int UNROLL, bool STREAM>
__global__ void __launch_bounds__(kThreads)
gps_kernel(const Chunk* __restrict__ chunks, GpsArgs a) {
    const Chunk c = chunks[blockIdx.x];
    const float* ob = a.outbox + c.begin;
    float* Th = a.Theta + c.begin;
    float* Mg = a.Mg + c.begin;
    float* ib = a.inbox + c.begin;
    const float eta = a.eta, beta = a.beta, omb = a.omb;
    uint32_t done = 0;
    if ((c.begin & 3ull) == 0) {
        const uint32_t nvec = c.count >> 2;
        for (uint32_t base = 0; base < nvec; base += kThreads * UNROLL) {
            float4 vd[UNROLL], vx[UNROLL], vm[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    vd[u] = ld4<STREAM>(ob + 4ull * v);
                    vx[u] = ld4<STREAM>(Th + 4ull * v);
                    vm[u] = ld4<STREAM>(Mg + 4ull * v);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    model_update(vx[u].x, vm[u].x, vd[u].x, eta, beta, omb);
                    model_update(vx[u].y, vm[u].y, vd[u].y, eta, beta, omb);
                    model_update(vx[u].z, vm[u].z, vd[u].z, eta, beta, omb);
                    model_update(vx[u].w, vm[u].w, vd[u].w, eta, beta, omb);
                    st4<STREAM>(Th + 4ull * v, vx[u]);
                    st4<STREAM>(Mg + 4ull * v, vm[u]);
                    st4<STREAM>(ib + 4ull * v, vx[u]);
                }
            }
        }
        done = nvec << 2;
    }
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads) {
        float x = Th[j], m = Mg[j];
        model_update(x, m, ob[j], eta, beta, omb);
        Th[j] = x;
        Mg[j] = m;
        ib[j] = x;
    }
}

// =====================================================================================================
// PULL: merge the received Theta_i and reset the anchor                          Alg. 1 lines 18-19
// =====================================================================================================
struct PullArgs {
    float* th;
    const float* inbox;
    float* anchor;
    float alpha, oma;
};

template <int UNROLL, bool STREAM>
__global__ void __launch_bounds__(kThreads)
pull_kernel(const Chunk* __restrict__ chunks, PullArgs a) {
    const Chunk c = chunks[blockIdx.x];
    float* th = a.th + c.begin;
    const float* ib = a.inbox + c.begin;
    float* an = a.anchor + c.begin;
    const float alpha = a.alpha, oma = a.oma;
    uint32_t done = 0;
    if ((c.begin & 3ull) == 0) {
        const uint32_t nvec = c.count >> 2;
        for (uint32_t base = 0; base < nvec; base += kThreads * UNROLL) {
            float4 vx[UNROLL], vy[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    vx[u] = ld4<STREAM>(th + 4ull * v);
                    vy[u] = ld4<STREAM>(ib + 4ull * v);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    float4 r;
                    r.x = merge(vx[u].x, vy[u].x, alpha, oma);
                    r.y = merge(vx[u].y, vy[u].y, alpha, oma);
                    r.z = merge(vx[u].z, vy[u].z, alpha, oma);
                    r.w = merge(vx[u].w, vy[u].w, alpha, oma);
                    st4<STREAM>(th + 4ull * v, r);
                    st4<STREAM>(an + 4ull * v, r);
                }
            }
        }
        done = nvec << 2;
    }
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads) {
        float r = merge(th[j], ib[j], alpha, oma);
        th[j] = r;
        an[j] = r;
    }
}

// =====================================================================================================
// Initialisation helpers and statistics finalisation
// =====================================================================================================
// theta0[w] <- cast(Theta_0) for bf16 worker copies (Alg. 1 line 7)
__global__ void cast_bf16_kernel(const float* __restrict__ src, uint16_t* __restrict__ dst, unsigned long long n) {
    unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    for (; i < n; i += stride) dst[i] = (uint16_t)bf16_narrow(src[i]);
}

// out[k] = sum of partial[c] over the chunks of tensor k, in a fixed order (one warp per tensor)
__global__ void stats_finalize_kernel(const double* __restrict__ partial, const uint32_t* __restrict__ tensor_chunk_begin,
                                      double* __restrict__ out, uint32_t n_tensors) {
    const uint32_t k = blockIdx.x;
    if (k >= n_tensors) return;
    const uint32_t b = tensor_chunk_begin[k], e = tensor_chunk_begin[k + 1];
    double v = 0.0;
    for (uint32_t c = b + threadIdx.x; c < e; c += 32) v += partial[c];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    if (threadIdx.x == 0) out[k] = v;
}

}  // namespace halos

// Fused, bandwidth-bound update kernels of the HALoS server path for sm_100a.
//
// One launch walks every tensor of the model through a chunk table built at context creation
// (the multi-tensor chunk scheduler): chunk c = {begin, count, tensor} is a run of `count`
// consecutive elements of the packed state starting at global element `begin`, never crossing a
// tensor boundary.  One CTA processes one chunk.  Inside a chunk every thread moves 128- or 256-bit
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

// Compile-time tuning knobs.  The defaults are the best of a sweep on B200 over threads {128, 256, 512},
// unroll {1, 2, 4, 8}, vector width {128, 256 bit}, evict-first hints {on, off} and chunk sizes
// 2048..65536 on a 162M-parameter buffer: 512 threads x one 256-bit vector per stream per thread
// (a CTA covers exactly one 4096-element chunk in a single batch of loads), no cache hints.
#ifndef HALOS_THREADS
#define HALOS_THREADS 512
#endif
#ifndef HALOS_UNROLL
#define HALOS_UNROLL 1
#endif
#ifndef HALOS_STREAM_HINT
#define HALOS_STREAM_HINT 0
#endif
#ifndef HALOS_VEC_ELEMS
#define HALOS_VEC_ELEMS 8
#endif
constexpr int kThreads = HALOS_THREADS;
constexpr int kVecElems = HALOS_VEC_ELEMS;   // elements per thread per access; chunks start on this boundary

// ---------------------------------------------------------------- element helpers
__device__ __forceinline__ void model_update(float& x, float& m, float d, float eta, float beta, float omb) {
    float m1 = __fmaf_rn(beta, m, d);
    float u = __fmaf_rn(beta, m1, __fmul_rn(omb, d));
    x = __fmaf_rn(eta, u, x);
    m = m1;
}
// Delayed-Nesterov step (optional optimizer; the reading is described in include/halos.h):
//   acc' = acc + d;  plain update: x' = x + (eps/n) d;  refresh: m' = beta m + acc'/n,
//   x' = x + eps (beta m' + d/n), acc' = 0.   inv_n = 1/n and eps_n = eps * inv_n are fp32 constants.
template <bool REFRESH>
__device__ __forceinline__ void delayed_nesterov(float& x, float& m, float& acc, float d, float eps, float beta,
                                                 float inv_n, float eps_n) {
    acc = __fadd_rn(acc, d);
    if (!REFRESH) {
        x = __fmaf_rn(eps_n, d, x);
    } else {
        float m1 = __fmaf_rn(beta, m, __fmul_rn(acc, inv_n));
        float u = __fmaf_rn(beta, m1, __fmul_rn(d, inv_n));
        x = __fmaf_rn(eps, u, x);
        m = m1;
        acc = 0.f;
    }
}
__device__ __forceinline__ float merge(float x, float y, float alpha, float oma) {
    return __fmaf_rn(alpha, y, __fmul_rn(oma, x));
}
__device__ __forceinline__ float bf16_widen(uint32_t h16) { return __uint_as_float(h16 << 16); }
__device__ __forceinline__ uint32_t bf16_narrow(float x) {
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x));  // round to nearest even
}

// ---------------------------------------------------------------- vector streaming access
// A thread moves VE consecutive elements per access: VE = 4 -> 128-bit (float4 / 4 x bf16 in 64 bits),
// VE = 8 -> 256-bit (ld/st.global.v8.f32, new with sm_100; 8 x bf16 in 128 bits).  Wider accesses
// halve the number of memory requests per byte.  State is touched once per event and the working
// set is far larger than L2, hence the evict-first (.cs) variants when STREAM is set.
template <int VE> struct FVec { float v[VE]; };

template <int VE, bool STREAM> __device__ __forceinline__ FVec<VE> ldf(const float* p);
template <int VE, bool STREAM> __device__ __forceinline__ void stf(float* p, const FVec<VE>& r);

template <> __device__ __forceinline__ FVec<4> ldf<4, true>(const float* p) {
    float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    return FVec<4>{{t.x, t.y, t.z, t.w}};
}
template <> __device__ __forceinline__ FVec<4> ldf<4, false>(const float* p) {
    float4 t = *reinterpret_cast<const float4*>(p);
    return FVec<4>{{t.x, t.y, t.z, t.w}};
}
template <> __device__ __forceinline__ void stf<4, true>(float* p, const FVec<4>& r) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(r.v[0], r.v[1], r.v[2], r.v[3]));
}
template <> __device__ __forceinline__ void stf<4, false>(float* p, const FVec<4>& r) {
    *reinterpret_cast<float4*>(p) = make_float4(r.v[0], r.v[1], r.v[2], r.v[3]);
}
template <> __device__ __forceinline__ FVec<8> ldf<8, true>(const float* p) {
    FVec<8> r;
    asm volatile("ld.global.cs.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
                 : "l"(p));
    return r;
}
template <> __device__ __forceinline__ FVec<8> ldf<8, false>(const float* p) {
    FVec<8> r;
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
                 : "l"(p));
    return r;
}
template <> __device__ __forceinline__ void stf<8, true>(float* p, const FVec<8>& r) {
    asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]),
                 "f"(r.v[3]), "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7])
                 : "memory");
}
template <> __device__ __forceinline__ void stf<8, false>(float* p, const FVec<8>& r) {
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]),
                 "f"(r.v[3]), "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7])
                 : "memory");
}

// bf16 rows: VE 16-bit patterns = VE/2 32-bit words
template <int VE, bool STREAM> __device__ __forceinline__ FVec<VE> ldh(const uint16_t* p);
template <int VE, bool STREAM> __device__ __forceinline__ void sth(uint16_t* p, const FVec<VE>& r);
template <int NW>
__device__ __forceinline__ void widen_words(const uint32_t* w, float* out) {
#pragma unroll
    for (int k = 0; k < NW; ++k) {
        out[2 * k] = bf16_widen(w[k] & 0xffffu);
        out[2 * k + 1] = bf16_widen(w[k] >> 16);
    }
}
template <int NW>
__device__ __forceinline__ void narrow_words(const float* in, uint32_t* w) {
#pragma unroll
    for (int k = 0; k < NW; ++k) w[k] = bf16_narrow(in[2 * k]) | (bf16_narrow(in[2 * k + 1]) << 16);
}
template <> __device__ __forceinline__ FVec<4> ldh<4, true>(const uint16_t* p) {
    uint2 t = __ldcs(reinterpret_cast<const uint2*>(p));
    uint32_t w[2] = {t.x, t.y};
    FVec<4> r;
    widen_words<2>(w, r.v);
    return r;
}
template <> __device__ __forceinline__ FVec<4> ldh<4, false>(const uint16_t* p) {
    uint2 t = *reinterpret_cast<const uint2*>(p);
    uint32_t w[2] = {t.x, t.y};
    FVec<4> r;
    widen_words<2>(w, r.v);
    return r;
}
template <> __device__ __forceinline__ FVec<8> ldh<8, true>(const uint16_t* p) {
    uint4 t = __ldcs(reinterpret_cast<const uint4*>(p));
    uint32_t w[4] = {t.x, t.y, t.z, t.w};
    FVec<8> r;
    widen_words<4>(w, r.v);
    return r;
}
template <> __device__ __forceinline__ FVec<8> ldh<8, false>(const uint16_t* p) {
    uint4 t = *reinterpret_cast<const uint4*>(p);
    uint32_t w[4] = {t.x, t.y, t.z, t.w};
    FVec<8> r;
    widen_words<4>(w, r.v);
    return r;
}
template <> __device__ __forceinline__ void sth<4, true>(uint16_t* p, const FVec<4>& r) {
    uint32_t w[2];
    narrow_words<2>(r.v, w);
    __stcs(reinterpret_cast<uint2*>(p), make_uint2(w[0], w[1]));
}
template <> __device__ __forceinline__ void sth<4, false>(uint16_t* p, const FVec<4>& r) {
    uint32_t w[2];
    narrow_words<2>(r.v, w);
    *reinterpret_cast<uint2*>(p) = make_uint2(w[0], w[1]);
}
template <> __device__ __forceinline__ void sth<8, true>(uint16_t* p, const FVec<8>& r) {
    uint32_t w[4];
    narrow_words<4>(r.v, w);
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
}
template <> __device__ __forceinline__ void sth<8, false>(uint16_t* p, const FVec<8>& r) {
    uint32_t w[4];
    narrow_words<4>(r.v, w);
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}

// worker-dtype traits: W = float (fp32 copies) or uint16_t (bf16 copies)
template <class W> struct WTraits;
template <> struct WTraits<float> {
    template <int VE, bool S> static __device__ __forceinline__ FVec<VE> load(const float* p) { return ldf<VE, S>(p); }
    template <int VE, bool S> static __device__ __forceinline__ void store(float* p, const FVec<VE>& v) { stf<VE, S>(p, v); }
    static __device__ __forceinline__ float load1(const float* p) { return *p; }
    static __device__ __forceinline__ void store1(float* p, float v) { *p = v; }
};
template <> struct WTraits<uint16_t> {
    template <int VE, bool S> static __device__ __forceinline__ FVec<VE> load(const uint16_t* p) { return ldh<VE, S>(p); }
    template <int VE, bool S> static __device__ __forceinline__ void store(uint16_t* p, const FVec<VE>& v) { sth<VE, S>(p, v); }
    static __device__ __forceinline__ float load1(const uint16_t* p) { return bf16_widen(*p); }
    static __device__ __forceinline__ void store1(uint16_t* p, float v) { *p = (uint16_t)bf16_narrow(v); }
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
    double* partial_theta;      // [n_chunks] sum theta_t^2 of the updated LPS model per chunk (STATS only)
    float eta, beta, omb;
};

template <int VE>
__device__ __forceinline__ float sumsq(const FVec<VE>& d, float acc) {
#pragma unroll
    for (int e = 0; e < VE; ++e) acc = fmaf(d.v[e], d.v[e], acc);
    return acc;
}

template <class W, bool PUSH, bool STATS, int UNROLL, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
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
    float acc_d = 0.f, acc_D = 0.f, acc_x = 0.f;

    // vector path: the chunk starts on a VE-element boundary of the packed state (bases are 256-byte
    // aligned) and the caller's theta_H pointer is aligned to one vector of its own type
    const bool vec_ok = ((c.begin % VE) == 0) && ((reinterpret_cast<uintptr_t>(h) % (VE * sizeof(W))) == 0);
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t base = 0; base < nvec; base += kThreads * UNROLL) {
            FVec<VE> vh[UNROLL], vs[UNROLL], vx[UNROLL], vm[UNROLL], va[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    const size_t o = (size_t)VE * v;
                    vh[u] = T::template load<VE, STREAM>(h + o);
                    vs[u] = T::template load<VE, STREAM>(s0 + o);
                    vx[u] = ldf<VE, STREAM>(th + o);
                    vm[u] = ldf<VE, STREAM>(ml + o);
                    if (PUSH) va[u] = ldf<VE, STREAM>(an + o);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    const size_t o = (size_t)VE * v;
                    FVec<VE> d;
#pragma unroll
                    for (int e = 0; e < VE; ++e) {
                        d.v[e] = __fsub_rn(vh[u].v[e], vs[u].v[e]);
                        model_update(vx[u].v[e], vm[u].v[e], d.v[e], eta, beta, omb);
                    }
                    stf<VE, STREAM>(th + o, vx[u]);
                    stf<VE, STREAM>(ml + o, vm[u]);
                    T::template store<VE, STREAM>(s0 + o, vx[u]);
                    if (STATS) {
                        acc_d = sumsq<VE>(d, acc_d);
                        acc_x = sumsq<VE>(vx[u], acc_x);
                    }
                    if (PUSH) {
                        FVec<VE> D;
#pragma unroll
                        for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx[u].v[e], va[u].v[e]);
                        stf<VE, STREAM>(ob + o, D);
                        if (STATS) acc_D = sumsq<VE>(D, acc_D);
                    }
                }
            }
        }
        done = nvec * VE;
    }
    // ragged tail (or a whole chunk whose pointers do not share the vector alignment): scalar
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads) {
        float d = __fsub_rn(T::load1(h + j), T::load1(s0 + j));
        float x = th[j], m = ml[j];
        model_update(x, m, d, eta, beta, omb);
        th[j] = x;
        ml[j] = m;
        T::store1(s0 + j, x);
        if (STATS) {
            acc_d = fmaf(d, d, acc_d);
            acc_x = fmaf(x, x, acc_x);
        }
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
        __syncthreads();
        double t3 = block_sum((double)acc_x, red);
        if (threadIdx.x == 0) a.partial_theta[blockIdx.x] = t3;
        if (PUSH) {
            __syncthreads();
            double t2 = block_sum((double)acc_D, red);
            if (threadIdx.x == 0) a.partial_Delta[blockIdx.x] = t2;
        }
    }
}

// =====================================================================================================
// ARRIVE x NB: NB consecutive arrivals at the same LPS (distinct workers) in ONE pass.  The LPS model
// and momentum are read and written once for the whole batch; per element the NB updates are applied
// in queue order in registers, so the result is bit-identical to NB single launches.  Traffic per
// batch: 8 + 8 (theta, m read + write) + NB x (2 w_b read + w_b write) instead of NB x (16 + 3 w_b).
// Only the last arrival of a batch may close a window of K (PUSH).  Batches of up to 4 run with the
// regular CTA size; 5..8 need ~150 registers per thread and run with 256-thread CTAs.
// =====================================================================================================
constexpr int kMaxBatch = 8;
constexpr int kMultiWideThreads = 256;   // CTA size of the multi-arrival kernel for batches of 3..8 (register budget)

template <class W>
struct ArriveMultiArgs {
    const W* h_flat[kMaxBatch];          // per arrival: flat result ...
    const W* const* h_ptrs[kMaxBatch];   // ... or per-tensor pointer table
    W* th0[kMaxBatch];                   // per arrival: that worker's start snapshot
    const unsigned long long* tensor_off;
    float* th;
    float* ml;
    const float* anchor;
    float* outbox;
    float eta, beta, omb;
};

template <class W, int NB, bool PUSH, bool STREAM, int VE, int TPB>
__global__ void __launch_bounds__(TPB, (NB <= 2 ? 1024 / TPB : (NB <= 4 ? 512 / TPB : 1)))
arrive_multi_kernel(const Chunk* __restrict__ chunks, ArriveMultiArgs<W> a) {
    using T = WTraits<W>;
    const Chunk c = chunks[blockIdx.x];
    const W* h[NB];
    W* s0[NB];
    bool vec_ok = (c.begin % VE) == 0;
#pragma unroll
    for (int j = 0; j < NB; ++j) {
        h[j] = a.h_flat[j] ? a.h_flat[j] + c.begin : a.h_ptrs[j][c.tensor] + (c.begin - a.tensor_off[c.tensor]);
        s0[j] = a.th0[j] + c.begin;
        vec_ok = vec_ok && ((reinterpret_cast<uintptr_t>(h[j]) % (VE * sizeof(W))) == 0);
    }
    float* th = a.th + c.begin;
    float* ml = a.ml + c.begin;
    const float* an = PUSH ? a.anchor + c.begin : nullptr;
    float* ob = PUSH ? a.outbox + c.begin : nullptr;
    const float eta = a.eta, beta = a.beta, omb = a.omb;
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t v = threadIdx.x; v < nvec; v += TPB) {
            const size_t o = (size_t)VE * v;
            FVec<VE> vh[NB], vs[NB], vx, vm, va;
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                vh[j] = T::template load<VE, STREAM>(h[j] + o);
                vs[j] = T::template load<VE, STREAM>(s0[j] + o);
            }
            vx = ldf<VE, STREAM>(th + o);
            vm = ldf<VE, STREAM>(ml + o);
            if (PUSH) va = ldf<VE, STREAM>(an + o);
#pragma unroll
            for (int j = 0; j < NB; ++j) {
#pragma unroll
                for (int e = 0; e < VE; ++e) {
                    const float d = __fsub_rn(vh[j].v[e], vs[j].v[e]);
                    model_update(vx.v[e], vm.v[e], d, eta, beta, omb);
                }
                T::template store<VE, STREAM>(s0[j] + o, vx);   // worker j restarts from the model after ITS update
            }
            stf<VE, STREAM>(th + o, vx);
            stf<VE, STREAM>(ml + o, vm);
            if (PUSH) {
                FVec<VE> D;
#pragma unroll
                for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx.v[e], va.v[e]);
                stf<VE, STREAM>(ob + o, D);
            }
        }
        done = nvec * VE;
    }
    for (uint32_t i = done + threadIdx.x; i < c.count; i += TPB) {
        float x = th[i], m = ml[i];
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            const float d = __fsub_rn(T::load1(h[j] + i), T::load1(s0[j] + i));
            model_update(x, m, d, eta, beta, omb);
            T::store1(s0[j] + i, x);
        }
        th[i] = x;
        ml[i] = m;
        if (PUSH) ob[i] = __fsub_rn(x, an[i]);
    }
}

// =====================================================================================================
// Delayed-Nesterov variants of ARRIVE and GPS.  A plain update touches theta and the accumulator
// (momentum is neither read nor written: same 16 + 3 w_b bytes per parameter as the paper's rule);
// a refresh update also reads and writes the momentum (+8 bytes).
// =====================================================================================================
template <class W>
struct ArriveDnArgs {
    const W* h_flat;
    const W* const* h_ptrs;
    const unsigned long long* tensor_off;
    W* th0;
    float* th;
    float* ml;
    float* acc;
    const float* anchor;
    float* outbox;
    float eps, beta, inv_n, eps_n;
};

template <class W, bool REFRESH, bool PUSH, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
arrive_dn_kernel(const Chunk* __restrict__ chunks, ArriveDnArgs<W> a) {
    using T = WTraits<W>;
    const Chunk c = chunks[blockIdx.x];
    const W* h = a.h_flat ? a.h_flat + c.begin : a.h_ptrs[c.tensor] + (c.begin - a.tensor_off[c.tensor]);
    W* s0 = a.th0 + c.begin;
    float* th = a.th + c.begin;
    float* ml = a.ml + c.begin;
    float* ac = a.acc + c.begin;
    const float* an = PUSH ? a.anchor + c.begin : nullptr;
    float* ob = PUSH ? a.outbox + c.begin : nullptr;
    const float eps = a.eps, beta = a.beta, inv_n = a.inv_n, eps_n = a.eps_n;
    const bool vec_ok = ((c.begin % VE) == 0) && ((reinterpret_cast<uintptr_t>(h) % (VE * sizeof(W))) == 0);
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t v = threadIdx.x; v < nvec; v += kThreads) {
            const size_t o = (size_t)VE * v;
            FVec<VE> vh = T::template load<VE, STREAM>(h + o);
            FVec<VE> vs = T::template load<VE, STREAM>(s0 + o);
            FVec<VE> vx = ldf<VE, STREAM>(th + o);
            FVec<VE> vc = ldf<VE, STREAM>(ac + o);
            FVec<VE> vm, va;
            if (REFRESH) vm = ldf<VE, STREAM>(ml + o);
            if (PUSH) va = ldf<VE, STREAM>(an + o);
#pragma unroll
            for (int e = 0; e < VE; ++e) {
                const float d = __fsub_rn(vh.v[e], vs.v[e]);
                float m = REFRESH ? vm.v[e] : 0.f;
                delayed_nesterov<REFRESH>(vx.v[e], m, vc.v[e], d, eps, beta, inv_n, eps_n);
                if (REFRESH) vm.v[e] = m;
            }
            stf<VE, STREAM>(th + o, vx);
            stf<VE, STREAM>(ac + o, vc);
            if (REFRESH) stf<VE, STREAM>(ml + o, vm);
            T::template store<VE, STREAM>(s0 + o, vx);
            if (PUSH) {
                FVec<VE> D;
#pragma unroll
                for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx.v[e], va.v[e]);
                stf<VE, STREAM>(ob + o, D);
            }
        }
        done = nvec * VE;
    }
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads) {
        const float d = __fsub_rn(T::load1(h + j), T::load1(s0 + j));
        float x = th[j], acc = ac[j], m = REFRESH ? ml[j] : 0.f;
        delayed_nesterov<REFRESH>(x, m, acc, d, eps, beta, inv_n, eps_n);
        th[j] = x;
        ac[j] = acc;
        if (REFRESH) ml[j] = m;
        T::store1(s0 + j, x);
        if (PUSH) ob[j] = __fsub_rn(x, an[j]);
    }
}

struct GpsDnArgs {
    const float* outbox;
    float* Theta;
    float* Mg;
    float* acc;
    float* inbox;
    float eps, beta, inv_n, eps_n;
};

template <bool REFRESH, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
gps_dn_kernel(const Chunk* __restrict__ chunks, GpsDnArgs a) {
    const Chunk c = chunks[blockIdx.x];
    const float* ob = a.outbox + c.begin;
    float* Th = a.Theta + c.begin;
    float* Mg = a.Mg + c.begin;
    float* ac = a.acc + c.begin;
    float* ib = a.inbox + c.begin;
    const float eps = a.eps, beta = a.beta, inv_n = a.inv_n, eps_n = a.eps_n;
    uint32_t done = 0;
    if ((c.begin % VE) == 0) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t v = threadIdx.x; v < nvec; v += kThreads) {
            const size_t o = (size_t)VE * v;
            FVec<VE> vd = ldf<VE, STREAM>(ob + o);
            FVec<VE> vx = ldf<VE, STREAM>(Th + o);
            FVec<VE> vc = ldf<VE, STREAM>(ac + o);
            FVec<VE> vm;
            if (REFRESH) vm = ldf<VE, STREAM>(Mg + o);
#pragma unroll
            for (int e = 0; e < VE; ++e) {
                float m = REFRESH ? vm.v[e] : 0.f;
                delayed_nesterov<REFRESH>(vx.v[e], m, vc.v[e], vd.v[e], eps, beta, inv_n, eps_n);
                if (REFRESH) vm.v[e] = m;
            }
            stf<VE, STREAM>(Th + o, vx);
            stf<VE, STREAM>(ac + o, vc);
            if (REFRESH) stf<VE, STREAM>(Mg + o, vm);
            stf<VE, STREAM>(ib + o, vx);
        }
        done = nvec * VE;
    }
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads) {
        float x = Th[j], acc = ac[j], m = REFRESH ? Mg[j] : 0.f;
        delayed_nesterov<REFRESH>(x, m, acc, ob[j], eps, beta, inv_n, eps_n);
        Th[j] = x;
        ac[j] = acc;
        if (REFRESH) Mg[j] = m;
        ib[j] = x;
    }
}

// =====================================================================================================
// ARRIVE x NB with the delayed-Nesterov optimizer: the model and the accumulator cross HBM once per
// batch; the momentum only if one of the batched updates is a refresh (bit j of refresh_mask).
// =====================================================================================================
template <class W>
struct ArriveMultiDnArgs {
    const W* h_flat[kMaxBatch];
    const W* const* h_ptrs[kMaxBatch];
    W* th0[kMaxBatch];
    const unsigned long long* tensor_off;
    float* th;
    float* ml;
    float* acc;
    const float* anchor;
    float* outbox;
    float eps, beta, inv_n, eps_n;
    uint32_t refresh_mask;
};

template <class W, int NB, bool ANYREF, bool PUSH, bool STREAM, int VE, int TPB>
__global__ void __launch_bounds__(TPB, (NB <= 2 ? 1024 / TPB : (NB <= 4 ? 512 / TPB : 1)))
arrive_multi_dn_kernel(const Chunk* __restrict__ chunks, ArriveMultiDnArgs<W> a) {
    using T = WTraits<W>;
    const Chunk c = chunks[blockIdx.x];
    const W* h[NB];
    W* s0[NB];
    bool vec_ok = (c.begin % VE) == 0;
#pragma unroll
    for (int j = 0; j < NB; ++j) {
        h[j] = a.h_flat[j] ? a.h_flat[j] + c.begin : a.h_ptrs[j][c.tensor] + (c.begin - a.tensor_off[c.tensor]);
        s0[j] = a.th0[j] + c.begin;
        vec_ok = vec_ok && ((reinterpret_cast<uintptr_t>(h[j]) % (VE * sizeof(W))) == 0);
    }
    float* th = a.th + c.begin;
    float* ml = a.ml + c.begin;
    float* ac = a.acc + c.begin;
    const float* an = PUSH ? a.anchor + c.begin : nullptr;
    float* ob = PUSH ? a.outbox + c.begin : nullptr;
    const float eps = a.eps, beta = a.beta, inv_n = a.inv_n, eps_n = a.eps_n;
    const uint32_t mask = a.refresh_mask;
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t v = threadIdx.x; v < nvec; v += TPB) {
            const size_t o = (size_t)VE * v;
            FVec<VE> vh[NB], vs[NB], vx, vc, vm, va;
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                vh[j] = T::template load<VE, STREAM>(h[j] + o);
                vs[j] = T::template load<VE, STREAM>(s0[j] + o);
            }
            vx = ldf<VE, STREAM>(th + o);
            vc = ldf<VE, STREAM>(ac + o);
            if (ANYREF) vm = ldf<VE, STREAM>(ml + o);
            if (PUSH) va = ldf<VE, STREAM>(an + o);
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                const bool refresh = ANYREF && ((mask >> j) & 1u);   // uniform over the grid
#pragma unroll
                for (int e = 0; e < VE; ++e) {
                    const float d = __fsub_rn(vh[j].v[e], vs[j].v[e]);
                    if (refresh) {
                        float m = vm.v[e];
                        delayed_nesterov<true>(vx.v[e], m, vc.v[e], d, eps, beta, inv_n, eps_n);
                        vm.v[e] = m;
                    } else {
                        float m = 0.f;
                        delayed_nesterov<false>(vx.v[e], m, vc.v[e], d, eps, beta, inv_n, eps_n);
                    }
                }
                T::template store<VE, STREAM>(s0[j] + o, vx);
            }
            stf<VE, STREAM>(th + o, vx);
            stf<VE, STREAM>(ac + o, vc);
            if (ANYREF) stf<VE, STREAM>(ml + o, vm);
            if (PUSH) {
                FVec<VE> D;
#pragma unroll
                for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx.v[e], va.v[e]);
                stf<VE, STREAM>(ob + o, D);
            }
        }
        done = nvec * VE;
    }
    for (uint32_t i = done + threadIdx.x; i < c.count; i += TPB) {
        float x = th[i], acc = ac[i], m = ANYREF ? ml[i] : 0.f;
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            const float d = __fsub_rn(T::load1(h[j] + i), T::load1(s0[j] + i));
            if (ANYREF && ((mask >> j) & 1u)) delayed_nesterov<true>(x, m, acc, d, eps, beta, inv_n, eps_n);
            else {
                float unused = 0.f;
                delayed_nesterov<false>(x, unused, acc, d, eps, beta, inv_n, eps_n);
            }
            T::store1(s0[j] + i, x);
        }
        th[i] = x;
        ac[i] = acc;
        if (ANYREF) ml[i] = m;
        if (PUSH) ob[i] = __fsub_rn(x, an[i]);
    }
}

// =====================================================================================================
// Materialised delta (HALOS_FLAG_MATERIALISE_DELTA): the worker-side subtraction of Alg. 1 line 25 runs
// when the result is handed over, delta (fp32) is kept in a context buffer, and the caller's theta_H is
// free again as soon as that kernel has been enqueued.  The LPS update then reads delta instead of
// theta_H and the old snapshot.  Same roundings as the fused path, hence the same bits.
// =====================================================================================================
template <class W>
struct DeltaArgs {
    const W* h_flat;
    const W* const* h_ptrs;
    const unsigned long long* tensor_off;
    const W* th0;
    float* delta;
};

template <class W, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
delta_kernel(const Chunk* __restrict__ chunks, DeltaArgs<W> a) {
    using T = WTraits<W>;
    const Chunk c = chunks[blockIdx.x];
    const W* h = a.h_flat ? a.h_flat + c.begin : a.h_ptrs[c.tensor] + (c.begin - a.tensor_off[c.tensor]);
    const W* s0 = a.th0 + c.begin;
    float* dl = a.delta + c.begin;
    const bool vec_ok = ((c.begin % VE) == 0) && ((reinterpret_cast<uintptr_t>(h) % (VE * sizeof(W))) == 0);
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t v = threadIdx.x; v < nvec; v += kThreads) {
            const size_t o = (size_t)VE * v;
            FVec<VE> vh = T::template load<VE, STREAM>(h + o);
            FVec<VE> vs = T::template load<VE, STREAM>(s0 + o);
            FVec<VE> d;
#pragma unroll
            for (int e = 0; e < VE; ++e) d.v[e] = __fsub_rn(vh.v[e], vs.v[e]);
            stf<VE, STREAM>(dl + o, d);
        }
        done = nvec * VE;
    }
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads)
        dl[j] = __fsub_rn(T::load1(h + j), T::load1(s0 + j));
}

template <class W>
struct ArriveDeltaArgs {
    const float* delta;
    W* th0;
    float* th;
    float* ml;
    const float* anchor;
    float* outbox;
    float eta, beta, omb;
};

template <class W, bool PUSH, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
arrive_delta_kernel(const Chunk* __restrict__ chunks, ArriveDeltaArgs<W> a) {
    using T = WTraits<W>;
    const Chunk c = chunks[blockIdx.x];
    const float* dl = a.delta + c.begin;
    W* s0 = a.th0 + c.begin;
    float* th = a.th + c.begin;
    float* ml = a.ml + c.begin;
    const float* an = PUSH ? a.anchor + c.begin : nullptr;
    float* ob = PUSH ? a.outbox + c.begin : nullptr;
    const float eta = a.eta, beta = a.beta, omb = a.omb;
    uint32_t done = 0;
    if ((c.begin % VE) == 0) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t v = threadIdx.x; v < nvec; v += kThreads) {
            const size_t o = (size_t)VE * v;
            FVec<VE> vd = ldf<VE, STREAM>(dl + o);
            FVec<VE> vx = ldf<VE, STREAM>(th + o);
            FVec<VE> vm = ldf<VE, STREAM>(ml + o);
            FVec<VE> va;
            if (PUSH) va = ldf<VE, STREAM>(an + o);
#pragma unroll
            for (int e = 0; e < VE; ++e) model_update(vx.v[e], vm.v[e], vd.v[e], eta, beta, omb);
            stf<VE, STREAM>(th + o, vx);
            stf<VE, STREAM>(ml + o, vm);
            T::template store<VE, STREAM>(s0 + o, vx);
            if (PUSH) {
                FVec<VE> D;
#pragma unroll
                for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx.v[e], va.v[e]);
                stf<VE, STREAM>(ob + o, D);
            }
        }
        done = nvec * VE;
    }
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads) {
        float x = th[j], m = ml[j];
        model_update(x, m, dl[j], eta, beta, omb);
        th[j] = x;
        ml[j] = m;
        T::store1(s0 + j, x);
        if (PUSH) ob[j] = __fsub_rn(x, an[j]);
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

template <bool STATS, int UNROLL, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads)
push_kernel(const Chunk* __restrict__ chunks, PushArgs a) {
    const Chunk c = chunks[blockIdx.x];
    const float* th = a.th + c.begin;
    const float* an = a.anchor + c.begin;
    float* ob = a.outbox + c.begin;
    float acc = 0.f;
    uint32_t done = 0;
    if ((c.begin % VE) == 0) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t base = 0; base < nvec; base += kThreads * UNROLL) {
            FVec<VE> vx[UNROLL], va[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    vx[u] = ldf<VE, STREAM>(th + (size_t)VE * v);
                    va[u] = ldf<VE, STREAM>(an + (size_t)VE * v);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    FVec<VE> D;
#pragma unroll
                    for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx[u].v[e], va[u].v[e]);
                    stf<VE, STREAM>(ob + (size_t)VE * v, D);
                    if (STATS) acc = sumsq<VE>(D, acc);
                }
            }
        }
        done = nvec * VE;
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

template <int UNROLL, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads)
gps_kernel(const Chunk* __restrict__ chunks, GpsArgs a) {
    const Chunk c = chunks[blockIdx.x];
    const float* ob = a.outbox + c.begin;
    float* Th = a.Theta + c.begin;
    float* Mg = a.Mg + c.begin;
    float* ib = a.inbox + c.begin;
    const float eta = a.eta, beta = a.beta, omb = a.omb;
    uint32_t done = 0;
    if ((c.begin % VE) == 0) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t base = 0; base < nvec; base += kThreads * UNROLL) {
            FVec<VE> vd[UNROLL], vx[UNROLL], vm[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    vd[u] = ldf<VE, STREAM>(ob + (size_t)VE * v);
                    vx[u] = ldf<VE, STREAM>(Th + (size_t)VE * v);
                    vm[u] = ldf<VE, STREAM>(Mg + (size_t)VE * v);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
#pragma unroll
                    for (int e = 0; e < VE; ++e) model_update(vx[u].v[e], vm[u].v[e], vd[u].v[e], eta, beta, omb);
                    stf<VE, STREAM>(Th + (size_t)VE * v, vx[u]);
                    stf<VE, STREAM>(Mg + (size_t)VE * v, vm[u]);
                    stf<VE, STREAM>(ib + (size_t)VE * v, vx[u]);
                }
            }
        }
        done = nvec * VE;
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

template <int UNROLL, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads)
pull_kernel(const Chunk* __restrict__ chunks, PullArgs a) {
    const Chunk c = chunks[blockIdx.x];
    float* th = a.th + c.begin;
    const float* ib = a.inbox + c.begin;
    float* an = a.anchor + c.begin;
    const float alpha = a.alpha, oma = a.oma;
    uint32_t done = 0;
    if ((c.begin % VE) == 0) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t base = 0; base < nvec; base += kThreads * UNROLL) {
            FVec<VE> vx[UNROLL], vy[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    vx[u] = ldf<VE, STREAM>(th + (size_t)VE * v);
                    vy[u] = ldf<VE, STREAM>(ib + (size_t)VE * v);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t v = base + u * kThreads + threadIdx.x;
                if (v < nvec) {
                    FVec<VE> r;
#pragma unroll
                    for (int e = 0; e < VE; ++e) r.v[e] = merge(vx[u].v[e], vy[u].v[e], alpha, oma);
                    stf<VE, STREAM>(th + (size_t)VE * v, r);
                    stf<VE, STREAM>(an + (size_t)VE * v, r);
                }
            }
        }
        done = nvec * VE;
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

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

// ---------------------------------------------------------------- statistics reduction
// Squared norms are reduced in a canonical order that does not depend on the CTA size or on how many
// arrivals a launch fuses, so that a fused launch reports the same fp64 sums, bit for bit, as the
// launches it replaces:
//   item     one vector of VE consecutive elements (vector path) or one element (scalar path); its value is
//            the fp32 sum of squares accumulated with fmaf from 0 in element order;
//   row      32 consecutive items of a chunk, summed in fp64 by a fixed shuffle tree (absent items count 0);
//   chunk    row sums added in fp64 in increasing row order (vector rows first, then scalar rows).
// A chunk of up to kStatMaxChunk elements has at most kStatRows rows.
constexpr int kStatRows = 256;
constexpr uint32_t kStatMaxChunk = kStatRows * 32;

__device__ __forceinline__ double row_sum(float item) {   // every lane of the warp calls it; valid in lane 0
    double v = (double)item;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}
template <int VE>
__device__ __forceinline__ float sumsq(const FVec<VE>& d) {
    float acc = 0.f;
#pragma unroll
    for (int e = 0; e < VE; ++e) acc = fmaf(d.v[e], d.v[e], acc);
    return acc;
}
// Adds the rows of quantity q in order; called by thread q (q < number of quantities) after a __syncthreads().
__device__ __forceinline__ double rows_total(const double* rows, uint32_t nrows) {
    double t = 0.0;
    for (uint32_t r = 0; r < nrows; ++r) t += rows[r];
    return t;
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
    __shared__ double srow[STATS ? 3 : 1][STATS ? kStatRows : 1];   // [delta^2, theta^2, Delta^2][row]
    const uint32_t lane = threadIdx.x & 31u, warp32 = threadIdx.x & ~31u;
    uint32_t nrv = 0;   // rows of the vector path

    // vector path: the chunk starts on a VE-element boundary of the packed state (bases are 256-byte
    // aligned) and the caller's theta_H pointer is aligned to one vector of its own type
    const bool vec_ok = ((c.begin % VE) == 0) && ((reinterpret_cast<uintptr_t>(h) % (VE * sizeof(W))) == 0);
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count / VE;
        nrv = (nvec + 31u) >> 5;
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
                float q_d = 0.f, q_x = 0.f, q_D = 0.f;
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
                        q_d = sumsq<VE>(d);
                        q_x = sumsq<VE>(vx[u]);
                    }
                    if (PUSH) {
                        FVec<VE> D;
#pragma unroll
                        for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx[u].v[e], va[u].v[e]);
                        stf<VE, STREAM>(ob + o, D);
                        if (STATS) q_D = sumsq<VE>(D);
                    }
                }
                if (STATS) {
                    const uint32_t vb = base + u * kThreads + warp32;   // first item of this warp's row
                    if (vb < nvec) {
                        const double r_d = row_sum(q_d), r_x = row_sum(q_x), r_D = PUSH ? row_sum(q_D) : 0.0;
                        if (lane == 0) {
                            srow[0][vb >> 5] = r_d;
                            srow[1][vb >> 5] = r_x;
                            if (PUSH) srow[2][vb >> 5] = r_D;
                        }
                    }
                }
            }
        }
        done = nvec * VE;
    }
    // ragged tail (or a whole chunk whose pointers do not share the vector alignment): scalar
    for (uint32_t jb = done + warp32; jb < c.count; jb += kThreads) {
        const uint32_t j = jb + lane;
        float q_d = 0.f, q_x = 0.f, q_D = 0.f;
        if (j < c.count) {
            float d = __fsub_rn(T::load1(h + j), T::load1(s0 + j));
            float x = th[j], m = ml[j];
            model_update(x, m, d, eta, beta, omb);
            th[j] = x;
            ml[j] = m;
            T::store1(s0 + j, x);
            if (STATS) {
                q_d = fmaf(d, d, 0.f);
                q_x = fmaf(x, x, 0.f);
            }
            if (PUSH) {
                float D = __fsub_rn(x, an[j]);
                ob[j] = D;
                if (STATS) q_D = fmaf(D, D, 0.f);
            }
        }
        if (STATS) {
            const uint32_t row = nrv + ((jb - done) >> 5);
            const double r_d = row_sum(q_d), r_x = row_sum(q_x), r_D = PUSH ? row_sum(q_D) : 0.0;
            if (lane == 0) {
                srow[0][row] = r_d;
                srow[1][row] = r_x;
                if (PUSH) srow[2][row] = r_D;
            }
        }
    }
    if (STATS) {
        __syncthreads();
        const uint32_t nrows = nrv + ((c.count - done + 31u) >> 5);
        if (threadIdx.x < (PUSH ? 3u : 2u)) {
            double* dst = threadIdx.x == 0 ? a.partial_delta : threadIdx.x == 1 ? a.partial_theta : a.partial_Delta;
            dst[blockIdx.x] = rows_total(srow[threadIdx.x], nrows);
        }
    }
}

// =====================================================================================================
// ARRIVE x NB: NB consecutive arrivals at the same LPS (distinct workers) in ONE pass.  The LPS model
// and momentum are read and written once for the whole batch; per element the NB updates are applied
// in queue order in registers, so the result is bit-identical to NB single launches.  Traffic per
// batch: 8 + 8 (theta, m read + write) + NB x (2 w_b read + w_b write) instead of NB x (16 + 3 w_b).
// Only the last arrival of a batch may close a window of K (PUSH).  Batches of 2 run with the regular CTA
// size (512 threads, 2 CTAs per SM); batches of 3..8 with 256-thread CTAs: 2 per SM up to 4 arrivals, and
// for 5..8 (150-240 registers with fp32 results) one per SM -- two for bf16 results, see multi_min_blocks.
// =====================================================================================================
constexpr int kMaxBatch = 8;
constexpr int kMultiWideThreads = 256;   // CTA size of the multi-arrival kernel for batches of 3..8 (register budget)

// Resident CTAs per SM the fused kernels are compiled for (it bounds the registers per thread).  Batches of
// 5..8 fp32 results keep 2 NB + 2 vectors of 32 B in flight per thread and saturate HBM with ONE CTA of 256
// threads per SM; bf16 results are half as wide, one CTA does not keep enough bytes in flight, so those
// kernels are compiled for two (128 registers, a few spilled to L1).
#ifndef HALOS_WIDE_MINBLOCKS_BF16
#define HALOS_WIDE_MINBLOCKS_BF16 2
#endif
// CTA size / resident CTAs of the delayed-Nesterov kernel for batches of 2 (one more stream than the paper rule).
#ifndef HALOS_DN2_THREADS
#define HALOS_DN2_THREADS 256
#endif
#ifndef HALOS_DN2_MINBLOCKS
#define HALOS_DN2_MINBLOCKS 3
#endif
#ifndef HALOS_WIDE_MINBLOCKS_BF16_STATS
#define HALOS_WIDE_MINBLOCKS_BF16_STATS 2
#endif
template <class W, int NB, int TPB, bool STATS = false>
constexpr int multi_min_blocks() {
    return NB <= 2 ? 1024 / TPB
                   : (NB <= 4 ? 512 / TPB : (sizeof(W) == 2 ? (STATS ? HALOS_WIDE_MINBLOCKS_BF16_STATS : HALOS_WIDE_MINBLOCKS_BF16) : 1));
}
template <int NB> constexpr int multi_threads() { return NB <= 2 ? kThreads : kMultiWideThreads; }
template <int NB> constexpr int multi_dn_threads() { return NB <= 2 ? HALOS_DN2_THREADS : kMultiWideThreads; }
template <class W, int NB, int TPB, bool STATS = false>
constexpr int multi_dn_min_blocks() {
    return NB <= 2 ? HALOS_DN2_MINBLOCKS : multi_min_blocks<W, NB, TPB, STATS>();
}

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
    double* partial_delta;               // [NB][n_chunks] sum delta^2 of arrival j per chunk   (STATS only)
    double* partial_theta;               // [NB][n_chunks] sum theta^2 right after arrival j    (STATS only)
    double* partial_Delta;               // [n_chunks]     sum Delta^2                          (STATS && PUSH)
    float eta, beta, omb;
};

// Statistics of a fused launch: quantity 2j = delta^2 of arrival j, 2j+1 = theta^2 after arrival j, 2 NB = Delta^2.
// Every lane of the warp calls this (lanes without an item pass 0).
__device__ __forceinline__ void stats_row_put(double* rows, uint32_t row, uint32_t lane, float item) {
    const double r = row_sum(item);
    if (lane == 0) rows[row] = r;
}
template <int NB, bool PUSH>
__device__ __forceinline__ void multi_stats_rows(double (*srow)[kStatRows + 1], uint32_t row, uint32_t lane,
                                                 const float* q_d, const float* q_x, float q_D) {
#pragma unroll
    for (int j = 0; j < NB; ++j) {
        stats_row_put(srow[2 * j], row, lane, q_d[j]);
        stats_row_put(srow[2 * j + 1], row, lane, q_x[j]);
    }
    if (PUSH) stats_row_put(srow[2 * NB], row, lane, q_D);
}
template <int NB, bool PUSH>
__device__ __forceinline__ void multi_stats_finish(double (*srow)[kStatRows + 1], uint32_t nrows, double* partial_delta,
                                                   double* partial_theta, double* partial_Delta) {
    __syncthreads();
    const uint32_t q = threadIdx.x;
    if (q < 2u * NB + (PUSH ? 1u : 0u)) {
        const double t = rows_total(srow[q], nrows);
        if (q == 2u * NB) partial_Delta[blockIdx.x] = t;
        else ((q & 1u) ? partial_theta : partial_delta)[(size_t)(q >> 1) * gridDim.x + blockIdx.x] = t;
    }
}

template <class W, int NB, bool PUSH, bool STATS, bool STREAM, int VE, int TPB>
__global__ void __launch_bounds__(TPB, (multi_min_blocks<W, NB, TPB, STATS>()))
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
    __shared__ double srow[STATS ? 2 * NB + 1 : 1][STATS ? kStatRows + 1 : 1];
    const uint32_t lane = threadIdx.x & 31u, warp32 = threadIdx.x & ~31u;
    uint32_t nrv = 0;
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count / VE;
        nrv = (nvec + 31u) >> 5;
        for (uint32_t vb = warp32; vb < nvec; vb += TPB) {   // a warp walks its rows of 32 vectors together
            const uint32_t v = vb + lane;
            float q_d[STATS ? NB : 1], q_x[STATS ? NB : 1], q_D = 0.f;   // this thread's items of the row (0 past the end)
            if (STATS) {
#pragma unroll
                for (int j = 0; j < NB; ++j) q_d[j] = q_x[j] = 0.f;
            }
            if (v < nvec) {
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
                    FVec<VE> d;
#pragma unroll
                    for (int e = 0; e < VE; ++e) {
                        d.v[e] = __fsub_rn(vh[j].v[e], vs[j].v[e]);
                        model_update(vx.v[e], vm.v[e], d.v[e], eta, beta, omb);
                    }
                    T::template store<VE, STREAM>(s0[j] + o, vx);   // worker j restarts from the model after ITS update
                    if (STATS) {
                        q_d[j] = sumsq<VE>(d);
                        q_x[j] = sumsq<VE>(vx);
                    }
                }
                stf<VE, STREAM>(th + o, vx);
                stf<VE, STREAM>(ml + o, vm);
                if (PUSH) {
                    FVec<VE> D;
#pragma unroll
                    for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx.v[e], va.v[e]);
                    stf<VE, STREAM>(ob + o, D);
                    if (STATS) q_D = sumsq<VE>(D);
                }
            }
            if constexpr (STATS) multi_stats_rows<NB, PUSH>(srow, vb >> 5, lane, q_d, q_x, q_D);   // after the stores are out
        }
        done = nvec * VE;
    }
    for (uint32_t ib = done + warp32; ib < c.count; ib += TPB) {
        const uint32_t i = ib + lane;
        float q_d[STATS ? NB : 1], q_x[STATS ? NB : 1], q_D = 0.f;
        if (STATS) {
#pragma unroll
            for (int j = 0; j < NB; ++j) q_d[j] = q_x[j] = 0.f;
        }
        if (i < c.count) {
            float x = th[i], m = ml[i];
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                const float d = __fsub_rn(T::load1(h[j] + i), T::load1(s0[j] + i));
                model_update(x, m, d, eta, beta, omb);
                T::store1(s0[j] + i, x);
                if (STATS) {
                    q_d[j] = fmaf(d, d, 0.f);
                    q_x[j] = fmaf(x, x, 0.f);
                }
            }
            th[i] = x;
            ml[i] = m;
            if (PUSH) {
                const float D = __fsub_rn(x, an[i]);
                ob[i] = D;
                if (STATS) q_D = fmaf(D, D, 0.f);
            }
        }
        if constexpr (STATS) multi_stats_rows<NB, PUSH>(srow, nrv + ((ib - done) >> 5), lane, q_d, q_x, q_D);
    }
    if constexpr (STATS)
        multi_stats_finish<NB, PUSH>(srow, nrv + ((c.count - done + 31u) >> 5), a.partial_delta, a.partial_theta, a.partial_Delta);
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
    double* partial_delta;   // statistics, as in ArriveArgs
    double* partial_Delta;
    double* partial_theta;
    float eps, beta, inv_n, eps_n;
};

template <class W, bool REFRESH, bool PUSH, bool STATS, bool STREAM, int VE>
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
    __shared__ double srow[STATS ? 3 : 1][STATS ? kStatRows : 1];
    const uint32_t lane = threadIdx.x & 31u, warp32 = threadIdx.x & ~31u;
    uint32_t nrv = 0;
    const bool vec_ok = ((c.begin % VE) == 0) && ((reinterpret_cast<uintptr_t>(h) % (VE * sizeof(W))) == 0);
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count / VE;
        nrv = (nvec + 31u) >> 5;
        for (uint32_t vb = warp32; vb < nvec; vb += kThreads) {
            const uint32_t v = vb + lane;
            float q_d = 0.f, q_x = 0.f, q_D = 0.f;
            if (v < nvec) {
                const size_t o = (size_t)VE * v;
                FVec<VE> vh = T::template load<VE, STREAM>(h + o);
                FVec<VE> vs = T::template load<VE, STREAM>(s0 + o);
                FVec<VE> vx = ldf<VE, STREAM>(th + o);
                FVec<VE> vc = ldf<VE, STREAM>(ac + o);
                FVec<VE> vm, va, d;
                if (REFRESH) vm = ldf<VE, STREAM>(ml + o);
                if (PUSH) va = ldf<VE, STREAM>(an + o);
#pragma unroll
                for (int e = 0; e < VE; ++e) {
                    d.v[e] = __fsub_rn(vh.v[e], vs.v[e]);
                    float m = REFRESH ? vm.v[e] : 0.f;
                    delayed_nesterov<REFRESH>(vx.v[e], m, vc.v[e], d.v[e], eps, beta, inv_n, eps_n);
                    if (REFRESH) vm.v[e] = m;
                }
                stf<VE, STREAM>(th + o, vx);
                stf<VE, STREAM>(ac + o, vc);
                if (REFRESH) stf<VE, STREAM>(ml + o, vm);
                T::template store<VE, STREAM>(s0 + o, vx);
                if (STATS) {
                    q_d = sumsq<VE>(d);
                    q_x = sumsq<VE>(vx);
                }
                if (PUSH) {
                    FVec<VE> D;
#pragma unroll
                    for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx.v[e], va.v[e]);
                    stf<VE, STREAM>(ob + o, D);
                    if (STATS) q_D = sumsq<VE>(D);
                }
            }
            if (STATS) {
                const double r_d = row_sum(q_d), r_x = row_sum(q_x), r_D = PUSH ? row_sum(q_D) : 0.0;
                if (lane == 0) {
                    srow[0][vb >> 5] = r_d;
                    srow[1][vb >> 5] = r_x;
                    if (PUSH) srow[2][vb >> 5] = r_D;
                }
            }
        }
        done = nvec * VE;
    }
    for (uint32_t jb = done + warp32; jb < c.count; jb += kThreads) {
        const uint32_t j = jb + lane;
        float q_d = 0.f, q_x = 0.f, q_D = 0.f;
        if (j < c.count) {
            const float d = __fsub_rn(T::load1(h + j), T::load1(s0 + j));
            float x = th[j], acc = ac[j], m = REFRESH ? ml[j] : 0.f;
            delayed_nesterov<REFRESH>(x, m, acc, d, eps, beta, inv_n, eps_n);
            th[j] = x;
            ac[j] = acc;
            if (REFRESH) ml[j] = m;
            T::store1(s0 + j, x);
            if (STATS) {
                q_d = fmaf(d, d, 0.f);
                q_x = fmaf(x, x, 0.f);
            }
            if (PUSH) {
                const float D = __fsub_rn(x, an[j]);
                ob[j] = D;
                if (STATS) q_D = fmaf(D, D, 0.f);
            }
        }
        if (STATS) {
            const uint32_t row = nrv + ((jb - done) >> 5);
            const double r_d = row_sum(q_d), r_x = row_sum(q_x), r_D = PUSH ? row_sum(q_D) : 0.0;
            if (lane == 0) {
                srow[0][row] = r_d;
                srow[1][row] = r_x;
                if (PUSH) srow[2][row] = r_D;
            }
        }
    }
    if (STATS) {
        __syncthreads();
        const uint32_t nrows = nrv + ((c.count - done + 31u) >> 5);
        if (threadIdx.x < (PUSH ? 3u : 2u)) {
            double* dst = threadIdx.x == 0 ? a.partial_delta : threadIdx.x == 1 ? a.partial_theta : a.partial_Delta;
            dst[blockIdx.x] = rows_total(srow[threadIdx.x], nrows);
        }
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
    double* partial_delta;   // statistics, as in ArriveMultiArgs
    double* partial_theta;
    double* partial_Delta;
    float eps, beta, inv_n, eps_n;
    uint32_t refresh_mask;
};

template <class W, int NB, bool ANYREF, bool PUSH, bool STATS, bool STREAM, int VE, int TPB>
__global__ void __launch_bounds__(TPB, (multi_dn_min_blocks<W, NB, TPB, STATS>()))
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
    __shared__ double srow[STATS ? 2 * NB + 1 : 1][STATS ? kStatRows + 1 : 1];
    const uint32_t lane = threadIdx.x & 31u, warp32 = threadIdx.x & ~31u;
    uint32_t nrv = 0;
    uint32_t done = 0;
    if (vec_ok) {
        const uint32_t nvec = c.count / VE;
        nrv = (nvec + 31u) >> 5;
        for (uint32_t vb = warp32; vb < nvec; vb += TPB) {
            const uint32_t v = vb + lane;
            float q_d[STATS ? NB : 1], q_x[STATS ? NB : 1], q_D = 0.f;
            if (STATS) {
#pragma unroll
                for (int j = 0; j < NB; ++j) q_d[j] = q_x[j] = 0.f;
            }
            if (v < nvec) {
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
                    FVec<VE> d;
#pragma unroll
                    for (int e = 0; e < VE; ++e) {
                        d.v[e] = __fsub_rn(vh[j].v[e], vs[j].v[e]);
                        if (refresh) {
                            float m = vm.v[e];
                            delayed_nesterov<true>(vx.v[e], m, vc.v[e], d.v[e], eps, beta, inv_n, eps_n);
                            vm.v[e] = m;
                        } else {
                            float m = 0.f;
                            delayed_nesterov<false>(vx.v[e], m, vc.v[e], d.v[e], eps, beta, inv_n, eps_n);
                        }
                    }
                    T::template store<VE, STREAM>(s0[j] + o, vx);
                    if (STATS) {
                        q_d[j] = sumsq<VE>(d);
                        q_x[j] = sumsq<VE>(vx);
                    }
                }
                stf<VE, STREAM>(th + o, vx);
                stf<VE, STREAM>(ac + o, vc);
                if (ANYREF) stf<VE, STREAM>(ml + o, vm);
                if (PUSH) {
                    FVec<VE> D;
#pragma unroll
                    for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx.v[e], va.v[e]);
                    stf<VE, STREAM>(ob + o, D);
                    if (STATS) q_D = sumsq<VE>(D);
                }
            }
            if constexpr (STATS) multi_stats_rows<NB, PUSH>(srow, vb >> 5, lane, q_d, q_x, q_D);
        }
        done = nvec * VE;
    }
    for (uint32_t ib = done + warp32; ib < c.count; ib += TPB) {
        const uint32_t i = ib + lane;
        float q_d[STATS ? NB : 1], q_x[STATS ? NB : 1], q_D = 0.f;
        if (STATS) {
#pragma unroll
            for (int j = 0; j < NB; ++j) q_d[j] = q_x[j] = 0.f;
        }
        if (i < c.count) {
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
                if (STATS) {
                    q_d[j] = fmaf(d, d, 0.f);
                    q_x[j] = fmaf(x, x, 0.f);
                }
            }
            th[i] = x;
            ac[i] = acc;
            if (ANYREF) ml[i] = m;
            if (PUSH) {
                const float D = __fsub_rn(x, an[i]);
                ob[i] = D;
                if (STATS) q_D = fmaf(D, D, 0.f);
            }
        }
        if constexpr (STATS) multi_stats_rows<NB, PUSH>(srow, nrv + ((ib - done) >> 5), lane, q_d, q_x, q_D);
    }
    if constexpr (STATS)
        multi_stats_finish<NB, PUSH>(srow, nrv + ((c.count - done + 31u) >> 5), a.partial_delta, a.partial_theta, a.partial_Delta);
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
    double* partial_delta;   // statistics, as in ArriveArgs
    double* partial_Delta;
    double* partial_theta;
};

template <class W, bool PUSH, bool STATS, bool STREAM, int VE>
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
    __shared__ double srow[STATS ? 3 : 1][STATS ? kStatRows : 1];
    const uint32_t lane = threadIdx.x & 31u, warp32 = threadIdx.x & ~31u;
    uint32_t nrv = 0;
    uint32_t done = 0;
    if ((c.begin % VE) == 0) {
        const uint32_t nvec = c.count / VE;
        nrv = (nvec + 31u) >> 5;
        for (uint32_t vb = warp32; vb < nvec; vb += kThreads) {
            const uint32_t v = vb + lane;
            float q_d = 0.f, q_x = 0.f, q_D = 0.f;
            if (v < nvec) {
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
                if (STATS) {
                    q_d = sumsq<VE>(vd);
                    q_x = sumsq<VE>(vx);
                }
                if (PUSH) {
                    FVec<VE> D;
#pragma unroll
                    for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx.v[e], va.v[e]);
                    stf<VE, STREAM>(ob + o, D);
                    if (STATS) q_D = sumsq<VE>(D);
                }
            }
            if (STATS) {
                const double r_d = row_sum(q_d), r_x = row_sum(q_x), r_D = PUSH ? row_sum(q_D) : 0.0;
                if (lane == 0) {
                    srow[0][vb >> 5] = r_d;
                    srow[1][vb >> 5] = r_x;
                    if (PUSH) srow[2][vb >> 5] = r_D;
                }
            }
        }
        done = nvec * VE;
    }
    for (uint32_t jb = done + warp32; jb < c.count; jb += kThreads) {
        const uint32_t j = jb + lane;
        float q_d = 0.f, q_x = 0.f, q_D = 0.f;
        if (j < c.count) {
            const float d = dl[j];
            float x = th[j], m = ml[j];
            model_update(x, m, d, eta, beta, omb);
            th[j] = x;
            ml[j] = m;
            T::store1(s0 + j, x);
            if (STATS) {
                q_d = fmaf(d, d, 0.f);
                q_x = fmaf(x, x, 0.f);
            }
            if (PUSH) {
                const float D = __fsub_rn(x, an[j]);
                ob[j] = D;
                if (STATS) q_D = fmaf(D, D, 0.f);
            }
        }
        if (STATS) {
            const uint32_t row = nrv + ((jb - done) >> 5);
            const double r_d = row_sum(q_d), r_x = row_sum(q_x), r_D = PUSH ? row_sum(q_D) : 0.0;
            if (lane == 0) {
                srow[0][row] = r_d;
                srow[1][row] = r_x;
                if (PUSH) srow[2][row] = r_D;
            }
        }
    }
    if (STATS) {
        __syncthreads();
        const uint32_t nrows = nrv + ((c.count - done + 31u) >> 5);
        if (threadIdx.x < (PUSH ? 3u : 2u)) {
            double* dst = threadIdx.x == 0 ? a.partial_delta : threadIdx.x == 1 ? a.partial_theta : a.partial_Delta;
            dst[blockIdx.x] = rows_total(srow[threadIdx.x], nrows);
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

template <bool STATS, int UNROLL, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads)
push_kernel(const Chunk* __restrict__ chunks, PushArgs a) {
    const Chunk c = chunks[blockIdx.x];
    const float* th = a.th + c.begin;
    const float* an = a.anchor + c.begin;
    float* ob = a.outbox + c.begin;
    __shared__ double srow[STATS ? kStatRows : 1];
    const uint32_t lane = threadIdx.x & 31u, warp32 = threadIdx.x & ~31u;
    uint32_t nrv = 0;
    uint32_t done = 0;
    if ((c.begin % VE) == 0) {
        const uint32_t nvec = c.count / VE;
        nrv = (nvec + 31u) >> 5;
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
                float q_D = 0.f;
                if (v < nvec) {
                    FVec<VE> D;
#pragma unroll
                    for (int e = 0; e < VE; ++e) D.v[e] = __fsub_rn(vx[u].v[e], va[u].v[e]);
                    stf<VE, STREAM>(ob + (size_t)VE * v, D);
                    if (STATS) q_D = sumsq<VE>(D);
                }
                if (STATS) {
                    const uint32_t vb = base + u * kThreads + warp32;
                    if (vb < nvec) {
                        const double r = row_sum(q_D);
                        if (lane == 0) srow[vb >> 5] = r;
                    }
                }
            }
        }
        done = nvec * VE;
    }
    for (uint32_t jb = done + warp32; jb < c.count; jb += kThreads) {
        const uint32_t j = jb + lane;
        float q_D = 0.f;
        if (j < c.count) {
            float D = __fsub_rn(th[j], an[j]);
            ob[j] = D;
            if (STATS) q_D = fmaf(D, D, 0.f);
        }
        if (STATS) {
            const double r = row_sum(q_D);
            if (lane == 0) srow[nrv + ((jb - done) >> 5)] = r;
        }
    }
    if (STATS) {
        __syncthreads();
        if (threadIdx.x == 0) a.partial_Delta[blockIdx.x] = rows_total(srow, nrv + ((c.count - done + 31u) >> 5));
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
// GPS + PULL for the same LPS in one pass: the GPS receives Delta_l, and the answer Theta_i is merged
// into that LPS at once (Alg. 1 lines 2-4 directly followed by lines 17-20 -- the order the event queue
// produces when the two messages are adjacent, as on a fast link).  Theta_i is still in registers when
// the merge needs it: 16 bytes read + 20 written per parameter instead of 24 + 16 for the two launches.
// The in-flight snapshot (inbox) is still written, so the state equals that of the two launches bit for bit.
// =====================================================================================================
struct GpsPullArgs {
    const float* outbox;
    float* Theta;
    float* Mg;
    float* acc;      // delayed Nesterov only
    float* inbox;
    float* th;       // theta of the LPS
    float* anchor;
    float eta, beta, omb;          // paper rule
    float inv_n, eps_n;            // delayed Nesterov (eta is its eps)
    float alpha, oma;
};

// MODE 0: the paper's ModelUpdate; 1: delayed Nesterov, plain update; 2: delayed Nesterov, refresh update
template <int MODE, bool STREAM, int VE>
__global__ void __launch_bounds__(kThreads)
gps_pull_kernel(const Chunk* __restrict__ chunks, GpsPullArgs a) {
    const Chunk c = chunks[blockIdx.x];
    const float* ob = a.outbox + c.begin;
    float* Th = a.Theta + c.begin;
    float* Mg = a.Mg + c.begin;
    float* ac = MODE ? a.acc + c.begin : nullptr;
    float* ib = a.inbox + c.begin;
    float* th = a.th + c.begin;
    float* an = a.anchor + c.begin;
    const float eta = a.eta, beta = a.beta, omb = a.omb, inv_n = a.inv_n, eps_n = a.eps_n, alpha = a.alpha, oma = a.oma;
    uint32_t done = 0;
    if ((c.begin % VE) == 0) {
        const uint32_t nvec = c.count / VE;
        for (uint32_t v = threadIdx.x; v < nvec; v += kThreads) {
            const size_t o = (size_t)VE * v;
            FVec<VE> vd = ldf<VE, STREAM>(ob + o);
            FVec<VE> vx = ldf<VE, STREAM>(Th + o);
            FVec<VE> vy = ldf<VE, STREAM>(th + o);
            FVec<VE> vm, vc;
            if (MODE != 1) vm = ldf<VE, STREAM>(Mg + o);
            if (MODE) vc = ldf<VE, STREAM>(ac + o);
#pragma unroll
            for (int e = 0; e < VE; ++e) {
                if (MODE == 0) model_update(vx.v[e], vm.v[e], vd.v[e], eta, beta, omb);
                else if (MODE == 1) {
                    float unused = 0.f;
                    delayed_nesterov<false>(vx.v[e], unused, vc.v[e], vd.v[e], eta, beta, inv_n, eps_n);
                } else delayed_nesterov<true>(vx.v[e], vm.v[e], vc.v[e], vd.v[e], eta, beta, inv_n, eps_n);
                vy.v[e] = merge(vy.v[e], vx.v[e], alpha, oma);
            }
            stf<VE, STREAM>(Th + o, vx);
            if (MODE != 1) stf<VE, STREAM>(Mg + o, vm);
            if (MODE) stf<VE, STREAM>(ac + o, vc);
            stf<VE, STREAM>(ib + o, vx);
            stf<VE, STREAM>(th + o, vy);
            stf<VE, STREAM>(an + o, vy);
        }
        done = nvec * VE;
    }
    for (uint32_t j = done + threadIdx.x; j < c.count; j += kThreads) {
        float x = Th[j], m = MODE != 1 ? Mg[j] : 0.f, acc = MODE ? ac[j] : 0.f;
        if (MODE == 0) model_update(x, m, ob[j], eta, beta, omb);
        else if (MODE == 1) delayed_nesterov<false>(x, m, acc, ob[j], eta, beta, inv_n, eps_n);
        else delayed_nesterov<true>(x, m, acc, ob[j], eta, beta, inv_n, eps_n);
        Th[j] = x;
        if (MODE != 1) Mg[j] = m;
        if (MODE) ac[j] = acc;
        ib[j] = x;
        const float r = merge(th[j], x, alpha, oma);
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

// Per-tensor statistics from per-chunk partial sums: one warp per (tensor, arrival of the launch, quantity)
// adds the chunks of its tensor in a fixed order.  Quantity 0 = delta^2, 1 = theta^2, 2 = Delta^2.
// The last arrival's sums go to `last` (what halos_stats reports for this LPS: [delta | Delta | theta][n_lps][nt]);
// every arrival's sums go to record seq[j] of the caller's log (3 nt doubles: delta | theta | Delta, the
// Delta part zero unless that arrival pushed) if the log has room for it.
struct StatsFinalizeArgs {
    const double* partial_delta;   // [nb][n_chunks]
    const double* partial_theta;   // [nb][n_chunks]
    const double* partial_Delta;   // [n_chunks]
    const uint32_t* tensor_chunk_begin;
    double* last;
    double* log;
    unsigned long long log_capacity;
    unsigned long long seq[kMaxBatch];   // log record of each arrival of the launch
    uint32_t n_chunks, n_tensors, n_lps, lps, nb;
    int push;                      // the last arrival formed Delta
};
__global__ void stats_finalize_kernel(StatsFinalizeArgs a) {
    const uint32_t k = blockIdx.x, j = blockIdx.y, q = blockIdx.z;
    const bool is_last = j + 1 == a.nb;
    const bool has_value = q < 2 || (is_last && a.push);
    double v = 0.0;
    if (has_value) {
        const double* partial = q == 0 ? a.partial_delta + (size_t)j * a.n_chunks
                              : q == 1 ? a.partial_theta + (size_t)j * a.n_chunks : a.partial_Delta;
        const uint32_t b = a.tensor_chunk_begin[k], e = a.tensor_chunk_begin[k + 1];
        for (uint32_t c = b + threadIdx.x; c < e; c += 32) v += partial[c];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    }
    if (threadIdx.x != 0) return;
    if (is_last && has_value) {
        const uint32_t what = q == 0 ? 0u : q == 1 ? 2u : 1u;
        a.last[((size_t)what * a.n_lps + a.lps) * a.n_tensors + k] = v;
    }
    if (a.log && a.seq[j] < a.log_capacity) a.log[((size_t)a.seq[j] * 3 + q) * a.n_tensors + k] = v;
}

// Delta^2 of a push launched on its own (halos_lps_push): out[k] = sum over the chunks of tensor k
__global__ void stats_finalize_push_kernel(const double* __restrict__ partial, const uint32_t* __restrict__ tensor_chunk_begin,
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

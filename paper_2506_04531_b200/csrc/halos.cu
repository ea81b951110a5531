// Host side of the HALoS server-path library: context, state machine of Algorithm 1, the
// multi-tensor chunk table, kernel launches, and the C ABI declared in include/halos.h.
#include "halos.h"
#include "halos_kernels.cuh"

#include <nvtx3/nvToolsExt.h>

#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

using namespace halos;

namespace {

constexpr uint32_t kDefaultChunkElems = kThreads * kVecElems * HALOS_UNROLL;  // one batch of loads per CTA: 4096
constexpr int kUnroll = HALOS_UNROLL;
constexpr bool kStream = HALOS_STREAM_HINT != 0;
constexpr int kVE = kVecElems;
constexpr int kStageSlots = 2;

thread_local std::string g_create_error;

struct LpsState {
    float *th = nullptr, *ml = nullptr, *anchor = nullptr, *outbox = nullptr, *inbox = nullptr;
    float* acc = nullptr;  // delayed Nesterov only
    uint64_t t = 0, t_last = 0, t_push = 0;
    uint64_t inbox_iter = 0;  // GPS iteration that produced the inbox content
    int phase = HALOS_IDLE;
};

enum { PEND_NONE = 0, PEND_FLAT = 1, PEND_PTRS = 2, PEND_STAGED = 3, PEND_DELTA = 4 };

struct WorkerState {
    void* th0 = nullptr;
    float* delta = nullptr;  // materialised displacement (HALOS_FLAG_MATERIALISE_DELTA only)
    uint32_t lps = 0;
    int pending = PEND_NONE;
    const void* flat = nullptr;
    int slot = -1;
    uint64_t round = 0;    // arrivals applied so far
    uint64_t sched_t = 0;  // LPS counter when last scheduled
    cudaEvent_t table_copied = nullptr;  // guards reuse of the pinned pointer-table slot
    cudaEvent_t snap_ready = nullptr;    // halos_worker_fetch_host: the snapshot to copy out has been written
    cudaEvent_t fetched = nullptr;       // ... and the copy to the host has read it
    bool fetch_outstanding = false;      // the next kernel that rewrites the snapshot must wait for `fetched`
    std::vector<uint8_t> vec_aligned;    // statistics contexts: per tensor, does the pending result allow the vector path
};

constexpr size_t kGuardBytes = 256;
struct GuardedBuffer {
    char* raw;       // start of the allocation: [guard | data (bytes) | slack + guard]
    size_t padded;   // data size rounded up to 256
    size_t bytes;    // data size
};

// An arrival whose counters are already advanced but whose kernel launch is deferred (multi-event fusion).
struct Deferred {
    uint32_t worker;
    const void* flat;   // NULL: per-tensor pointer table of that worker
    bool refresh;       // delayed Nesterov: this update refreshes the momentum (decided when it was accounted for)
    uint64_t seq;       // record of this arrival in the statistics log
};

struct TimedLaunch {
    cudaEvent_t a, b;
    int kind;
    uint32_t events;           // events of the trace this launch carried out
    uint32_t bytes_per_param;  // its algorithmic traffic per parameter
};

}  // namespace

struct halos_ctx {
    halos_config cfg;
    uint64_t P = 0;
    uint32_t wb = 4;  // bytes per worker-copy element
    std::vector<uint64_t> tensor_numel, tensor_off;
    std::vector<uint32_t> worker_lps;
    std::vector<Chunk> chunks;
    std::vector<uint32_t> tensor_chunk_begin;
    cudaStream_t stream = nullptr;
    cudaStream_t copy_stream = nullptr;
    cudaStream_t d2h_stream = nullptr;   // device-to-host copies of worker snapshots (created on first use)

    Chunk* d_chunks = nullptr;
    Chunk* d_chunks_rev = nullptr;  // the same table in reverse order
    bool flip = false;              // direction of the next launch
    unsigned long long* d_tensor_off = nullptr;
    uint32_t* d_tensor_chunk_begin = nullptr;
    const void** d_ptr_tables = nullptr;  // [n_workers][n_tensors]
    const void** h_ptr_tables = nullptr;  // pinned mirror
    double *d_partial_delta = nullptr, *d_partial_Delta = nullptr, *d_partial_theta = nullptr;
    double* d_stats = nullptr;  // [3][n_lps][n_tensors]
    double* stats_log = nullptr;        // caller-owned device log of per-arrival statistics (halos_stats_log)
    uint64_t stats_log_capacity = 0;    // in records of 3 n_tensors doubles
    uint64_t stats_seq = 0;             // arrivals accounted for since the log was attached

    float *Theta = nullptr, *Mg = nullptr;
    float* acc_g = nullptr;  // delayed Nesterov only
    uint64_t gps_iter = 0;
    std::vector<LpsState> lps;
    std::vector<WorkerState> workers;

    void* stage[kStageSlots] = {nullptr, nullptr};
    cudaEvent_t stage_ready[kStageSlots] = {nullptr, nullptr};
    cudaEvent_t stage_free[kStageSlots] = {nullptr, nullptr};
    int stage_owner[kStageSlots] = {-1, -1};
    int stage_next = 0;

    std::vector<std::vector<Deferred>> deferred;  // per LPS: arrivals accounted for, not yet launched
    std::vector<void*> owned;  // device allocations made through the allocator
    std::vector<GuardedBuffer> guards;
    uint64_t launches = 0;
    uint64_t batched_arrivals = 0;  // arrivals that ran inside a multi-arrival launch
    uint64_t multi_launches = 0;
    bool timing = false;
    std::vector<TimedLaunch> timed;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> event_pool;
    std::string err;
};

namespace {

int fail(halos_ctx* c, int status, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (c) c->err = buf;
    else g_create_error = buf;
    return status;
}

#define CU(c, call)                                                                                   \
    do {                                                                                              \
        cudaError_t e_ = (call);                                                                      \
        if (e_ != cudaSuccess) return fail((c), HALOS_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

void* dev_alloc(halos_ctx* c, size_t bytes) {
    if (bytes == 0) bytes = 256;
    void* p = nullptr;
    if (c->cfg.alloc) {
        p = c->cfg.alloc(bytes, c->cfg.alloc_user);
    } else if (cudaMalloc(&p, bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        p = nullptr;
    }
    if (p) c->owned.push_back(p);
    return p;
}

void release(halos_ctx* c) {
    cudaStreamSynchronize(c->stream);
    if (c->copy_stream) {
        cudaStreamSynchronize(c->copy_stream);
        cudaStreamDestroy(c->copy_stream);
    }
    if (c->d2h_stream) {
        cudaStreamSynchronize(c->d2h_stream);
        cudaStreamDestroy(c->d2h_stream);
    }
    for (void* p : c->owned) {
        if (c->cfg.free_ && c->cfg.alloc) c->cfg.free_(p, c->cfg.alloc_user);
        else cudaFree(p);
    }
    c->owned.clear();
    if (c->h_ptr_tables) cudaFreeHost((void*)c->h_ptr_tables);
    for (auto& w : c->workers) {
        if (w.table_copied) cudaEventDestroy(w.table_copied);
        if (w.snap_ready) cudaEventDestroy(w.snap_ready);
        if (w.fetched) cudaEventDestroy(w.fetched);
    }
    for (int s = 0; s < kStageSlots; ++s) {
        if (c->stage_ready[s]) cudaEventDestroy(c->stage_ready[s]);
        if (c->stage_free[s]) cudaEventDestroy(c->stage_free[s]);
    }
    for (auto& t : c->timed) {
        cudaEventDestroy(t.a);
        cudaEventDestroy(t.b);
    }
    for (auto& e : c->event_pool) {
        cudaEventDestroy(e.first);
        cudaEventDestroy(e.second);
    }
    (void)cudaGetLastError();
}

// The chunk table: each tensor is cut into an unaligned head (fewer than kVecElems elements, so that
// everything after it starts on a vector boundary of the packed state), full chunks, and a tail.
void build_chunks(halos_ctx* c, uint32_t chunk_elems) {
    c->chunks.clear();
    c->tensor_chunk_begin.assign(c->tensor_numel.size() + 1, 0);
    for (size_t k = 0; k < c->tensor_numel.size(); ++k) {
        c->tensor_chunk_begin[k] = (uint32_t)c->chunks.size();
        uint64_t pos = c->tensor_off[k], end = c->tensor_off[k] + c->tensor_numel[k];
        uint64_t head = (kVE - (pos % kVE)) % kVE;
        if (head && pos < end) {
            uint64_t n = head < end - pos ? head : end - pos;
            c->chunks.push_back(Chunk{pos, (uint32_t)n, (uint32_t)k});
            pos += n;
        }
        while (pos < end) {
            uint64_t n = end - pos < chunk_elems ? end - pos : chunk_elems;
            c->chunks.push_back(Chunk{pos, (uint32_t)n, (uint32_t)k});
            pos += n;
        }
    }
    c->tensor_chunk_begin[c->tensor_numel.size()] = (uint32_t)c->chunks.size();
}

// Brackets one kernel launch: an NVTX range named after the kernel kind (visible to profilers, free
// otherwise) and, while timing is enabled, a pair of CUDA events on the context's stream.
const char* const kKindNames[HALOS_K_COUNT] = {"halos:arrive", "halos:arrive+push", "halos:push", "halos:gps",
                                               "halos:pull", "halos:arrive_multi", "halos:gps+pull"};
// Chunk table of the next launch.  Consecutive launches walk the buffers in opposite directions, so that
// a launch starts on the lines its predecessor touched last, which are still in L2 (worth 1-3% on
// buffers several times the size of L2).  Statistics index their partial sums by table position and
// always use the forward table.
const Chunk* next_table(halos_ctx* c) {
    if (c->cfg.flags & HALOS_FLAG_STATS) return c->d_chunks;
    c->flip = !c->flip;
    return c->flip ? c->d_chunks : c->d_chunks_rev;
}

struct Timer {
    halos_ctx* c;
    cudaEvent_t a = nullptr, b = nullptr;
    int kind;
    uint32_t events, bpp;
    // events: trace events the launch carries out; bpp: bytes it must move per parameter (each live buffer read
    // once and written once)
    Timer(halos_ctx* c_, int kind_, uint32_t events_, uint32_t bpp_) : c(c_), kind(kind_), events(events_), bpp(bpp_) {
        nvtxRangePushA(kKindNames[kind]);
        if (!c->timing) return;
        if (!c->event_pool.empty()) {
            a = c->event_pool.back().first;
            b = c->event_pool.back().second;
            c->event_pool.pop_back();
        } else if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) {
            a = b = nullptr;
            (void)cudaGetLastError();
            return;
        }
        cudaEventRecord(a, c->stream);
    }
    void stop() {
        nvtxRangePop();
        if (!a) return;
        cudaEventRecord(b, c->stream);
        c->timed.push_back(TimedLaunch{a, b, kind, events, bpp});
    }
};

// Launch helpers pick the template instance from run-time booleans.
#define HALOS_PICK2(b0, b1, CALL)                     \
    do {                                              \
        if (b0) {                                     \
            if (b1) { CALL(true, true); }             \
            else { CALL(true, false); }               \
        } else {                                      \
            if (b1) { CALL(false, true); }            \
            else { CALL(false, false); }              \
        }                                             \
    } while (0)

inline bool stats_on(const halos_ctx* c) { return (c->cfg.flags & HALOS_FLAG_STATS) != 0; }

// A kernel is about to rewrite this worker's snapshot: it must not overtake a copy of the old one to the host.
int wait_fetch(halos_ctx* c, WorkerState& w) {
    if (!w.fetch_outstanding) return HALOS_OK;
    CU(c, cudaStreamWaitEvent(c->stream, w.fetched, 0));
    w.fetch_outstanding = false;
    return HALOS_OK;
}

template <class W>
int launch_arrive_dn(halos_ctx* c, LpsState& s, WorkerState& w, uint32_t widx, bool push, const void* flat, int refresh_known) {
    ArriveDnArgs<W> a;
    a.h_flat = (const W*)flat;
    a.h_ptrs = flat ? nullptr : (const W* const*)(c->d_ptr_tables + (size_t)widx * c->tensor_numel.size());
    a.tensor_off = c->d_tensor_off;
    a.th0 = (W*)w.th0;
    a.th = s.th;
    a.ml = s.ml;
    a.acc = s.acc;
    a.anchor = s.anchor;
    a.outbox = s.outbox;
    a.partial_delta = c->d_partial_delta;
    a.partial_Delta = c->d_partial_Delta;
    a.partial_theta = c->d_partial_theta;
    a.eps = c->cfg.eta_l;
    a.beta = c->cfg.beta_l;
    a.inv_n = 1.0f / (float)c->cfg.delay_l;
    a.eps_n = c->cfg.eta_l * a.inv_n;
    // refresh_known < 0: the launch precedes the counter update, so this is update number s.t + 1
    const bool refresh = refresh_known >= 0 ? refresh_known != 0 : ((s.t + 1) % c->cfg.delay_l) == 0;
    const dim3 grid((unsigned)c->chunks.size()), block(kThreads);
    if (grid.x == 0) return HALOS_OK;
    Timer tm(c, push ? HALOS_K_ARRIVE_PUSH : HALOS_K_ARRIVE, 1, 16 + 3 * c->wb + (push ? 8 : 0) + (refresh ? 8 : 0));
    const Chunk* table = next_table(c);
    if (stats_on(c)) {
#define CALL(R, P) arrive_dn_kernel<W, R, P, true, kStream, kVE><<<grid, block, 0, c->stream>>>(table, a)
        HALOS_PICK2(refresh, push, CALL);
#undef CALL
    } else {
#define CALL(R, P) arrive_dn_kernel<W, R, P, false, kStream, kVE><<<grid, block, 0, c->stream>>>(table, a)
        HALOS_PICK2(refresh, push, CALL);
#undef CALL
    }
    tm.stop();
    c->launches++;
    CU(c, cudaGetLastError());
    return HALOS_OK;
}

template <class W>
int launch_arrive(halos_ctx* c, LpsState& s, WorkerState& w, uint32_t widx, bool push, const void* flat, int refresh_known = -1) {
    {
        int rw = wait_fetch(c, w);
        if (rw != HALOS_OK) return rw;
    }
    if (c->cfg.optimizer == HALOS_OPT_DELAYED_NESTEROV) return launch_arrive_dn<W>(c, s, w, widx, push, flat, refresh_known);
    const bool stats = stats_on(c);
    if (w.pending == PEND_DELTA) {
        ArriveDeltaArgs<W> d{w.delta, (W*)w.th0, s.th, s.ml, s.anchor, s.outbox, c->cfg.eta_l, c->cfg.beta_l, 1.0f - c->cfg.beta_l,
                             c->d_partial_delta, c->d_partial_Delta, c->d_partial_theta};
        const dim3 grid((unsigned)c->chunks.size()), block(kThreads);
        if (grid.x == 0) return HALOS_OK;
        Timer tm(c, push ? HALOS_K_ARRIVE_PUSH : HALOS_K_ARRIVE, 1, 20 + c->wb + (push ? 8 : 0));   // reads delta, not theta_H and theta_0
        const Chunk* table = next_table(c);
#define CALL(P, S) arrive_delta_kernel<W, P, S, kStream, kVE><<<grid, block, 0, c->stream>>>(table, d)
        HALOS_PICK2(push, stats, CALL);
#undef CALL
        tm.stop();
        c->launches++;
        CU(c, cudaGetLastError());
        return HALOS_OK;
    }
    ArriveArgs<W> a;
    a.h_flat = (const W*)flat;
    a.h_ptrs = flat ? nullptr : (const W* const*)(c->d_ptr_tables + (size_t)widx * c->tensor_numel.size());
    a.tensor_off = c->d_tensor_off;
    a.th0 = (W*)w.th0;
    a.th = s.th;
    a.ml = s.ml;
    a.anchor = s.anchor;
    a.outbox = s.outbox;
    a.partial_delta = c->d_partial_delta;
    a.partial_Delta = c->d_partial_Delta;
    a.partial_theta = c->d_partial_theta;
    a.eta = c->cfg.eta_l;
    a.beta = c->cfg.beta_l;
    a.omb = 1.0f - c->cfg.beta_l;
    const dim3 grid((unsigned)c->chunks.size()), block(kThreads);
    if (grid.x == 0) return HALOS_OK;
    Timer tm(c, push ? HALOS_K_ARRIVE_PUSH : HALOS_K_ARRIVE, 1, 16 + 3 * c->wb + (push ? 8 : 0));
    const Chunk* table = next_table(c);
#define CALL(P, S) arrive_kernel<W, P, S, kUnroll, kStream, kVE><<<grid, block, 0, c->stream>>>(table, a)
    HALOS_PICK2(push, stats, CALL);
#undef CALL
    tm.stop();
    c->launches++;
    CU(c, cudaGetLastError());
    return HALOS_OK;
}

// Per-tensor statistics of the nb arrivals of the launch just enqueued; seq[j] = log record of arrival j.
int finalize_stats(halos_ctx* c, uint32_t lps, uint32_t nb, bool push, const uint64_t* seq) {
    StatsFinalizeArgs a;
    a.partial_delta = c->d_partial_delta;
    a.partial_theta = c->d_partial_theta;
    a.partial_Delta = c->d_partial_Delta;
    a.tensor_chunk_begin = c->d_tensor_chunk_begin;
    a.last = c->d_stats;
    a.log = c->stats_log;
    a.log_capacity = c->stats_log_capacity;
    for (uint32_t j = 0; j < (uint32_t)kMaxBatch; ++j) a.seq[j] = j < nb ? seq[j] : ~0ull;
    a.n_chunks = (uint32_t)c->chunks.size();
    a.n_tensors = (uint32_t)c->tensor_numel.size();
    a.n_lps = c->cfg.n_lps;
    a.lps = lps;
    a.nb = nb;
    a.push = push ? 1 : 0;
    stats_finalize_kernel<<<dim3(a.n_tensors, nb, 3), 32, 0, c->stream>>>(a);
    c->launches++;
    CU(c, cudaGetLastError());
    return HALOS_OK;
}

// delta[w] <- theta_H - theta0[w] now (Alg. 1 line 25 as a kernel of its own); flat == NULL: pointer table of w.
template <class W>
int launch_delta_t(halos_ctx* c, uint32_t worker, const void* flat) {
    WorkerState& w = c->workers[worker];
    DeltaArgs<W> a;
    a.h_flat = (const W*)flat;
    a.h_ptrs = flat ? nullptr : (const W* const*)(c->d_ptr_tables + (size_t)worker * c->tensor_numel.size());
    a.tensor_off = c->d_tensor_off;
    a.th0 = (const W*)w.th0;
    a.delta = w.delta;
    const dim3 grid((unsigned)c->chunks.size()), block(kThreads);
    if (grid.x) delta_kernel<W, kStream, kVE><<<grid, block, 0, c->stream>>>(next_table(c), a);
    c->launches++;
    CU(c, cudaGetLastError());
    return HALOS_OK;
}
int launch_delta(halos_ctx* c, uint32_t worker, const void* flat) {
    return c->wb == 4 ? launch_delta_t<float>(c, worker, flat) : launch_delta_t<uint16_t>(c, worker, flat);
}

// Host-side part of an arrival (Alg. 1 lines 10 and 13): argument/state checks and counter updates.
// *due = this arrival completes a window of K; *push = the caller wants Delta formed with it.
// The part of the check that does not need a registered result (the replay driver runs it BEFORE it asks
// the producer for one, so that a refused event leaves no borrowed pointer behind).
int arrival_check(halos_ctx* c, uint32_t lps, uint32_t worker, bool fuse_push, bool* due, bool* push) {
    if (lps >= c->cfg.n_lps || worker >= c->cfg.n_workers) return fail(c, HALOS_ERR_INVALID_ARG, "lps/worker out of range");
    WorkerState& w = c->workers[worker];
    if (w.lps != lps) return fail(c, HALOS_ERR_INVALID_ARG, "worker %u does not belong to LPS %u", worker, lps);
    LpsState& s = c->lps[lps];
    *due = (s.t + 1 - s.t_last == c->cfg.K);
    *push = fuse_push && *due;
    if (*push && s.phase != HALOS_IDLE) return fail(c, HALOS_ERR_BAD_STATE, "LPS %u: push due while a round trip is in flight", lps);
    return HALOS_OK;
}

int apply_check(halos_ctx* c, uint32_t lps, uint32_t worker, bool fuse_push, bool* due, bool* push) {
    int rc = arrival_check(c, lps, worker, fuse_push, due, push);
    if (rc != HALOS_OK) return rc;
    if (c->workers[worker].pending == PEND_NONE) return fail(c, HALOS_ERR_BAD_STATE, "worker %u has no pending result", worker);
    return HALOS_OK;
}

void apply_commit(halos_ctx* c, uint32_t lps, uint32_t worker, bool push) {
    WorkerState& w = c->workers[worker];
    LpsState& s = c->lps[lps];
    w.pending = PEND_NONE;
    w.flat = nullptr;
    w.slot = -1;
    w.round += 1;
    s.t += 1;
    w.sched_t = s.t;
    if (push) {
        s.phase = HALOS_PUSHED;
        s.t_push = s.t;
    }
}

// lps_apply with an optional fused push; shared by the C entry point and the replay driver.
int apply_impl(halos_ctx* c, uint32_t lps, uint32_t worker, bool fuse_push, int* push_due) {
    bool due = false, push = false;
    int rc = apply_check(c, lps, worker, fuse_push, &due, &push);
    if (rc != HALOS_OK) return rc;
    WorkerState& w = c->workers[worker];
    LpsState& s = c->lps[lps];
    CU(c, cudaSetDevice(c->cfg.device));
    const void* flat = nullptr;
    if (w.pending == PEND_FLAT) flat = w.flat;
    if (w.pending == PEND_STAGED) {
        flat = c->stage[w.slot];
        CU(c, cudaStreamWaitEvent(c->stream, c->stage_ready[w.slot], 0));
    }
    rc = c->wb == 4 ? launch_arrive<float>(c, s, w, worker, push, flat)
                    : launch_arrive<uint16_t>(c, s, w, worker, push, flat);
    if (rc != HALOS_OK) return rc;
    if (w.pending == PEND_STAGED) {
        CU(c, cudaEventRecord(c->stage_free[w.slot], c->stream));
        c->stage_owner[w.slot] = -1;
    }
    if (stats_on(c) && (rc = finalize_stats(c, lps, 1, push, &c->stats_seq)) != HALOS_OK) return rc;
    c->stats_seq += 1;
    apply_commit(c, lps, worker, push);
    if (push_due) *push_due = due ? 1 : 0;
    return HALOS_OK;
}

// ---- batched arrivals (multi-event fusion) -------------------------------------------------------

template <class W, int NB>
int launch_arrive_multi_dn(halos_ctx* c, LpsState& s, const Deferred* d, bool push) {
    ArriveMultiDnArgs<W> a;
    const size_t nt = c->tensor_numel.size();
    a.refresh_mask = 0;
    for (int j = 0; j < kMaxBatch; ++j) {
        const int k = j < NB ? j : 0;
        a.h_flat[j] = (const W*)d[k].flat;
        a.h_ptrs[j] = d[k].flat ? nullptr : (const W* const*)(c->d_ptr_tables + (size_t)d[k].worker * nt);
        a.th0[j] = (W*)c->workers[d[k].worker].th0;
        if (j < NB && d[j].refresh) a.refresh_mask |= 1u << j;
    }
    a.tensor_off = c->d_tensor_off;
    a.th = s.th;
    a.ml = s.ml;
    a.acc = s.acc;
    a.anchor = s.anchor;
    a.outbox = s.outbox;
    a.partial_delta = c->d_partial_delta;
    a.partial_theta = c->d_partial_theta;
    a.partial_Delta = c->d_partial_Delta;
    a.eps = c->cfg.eta_l;
    a.beta = c->cfg.beta_l;
    a.inv_n = 1.0f / (float)c->cfg.delay_l;
    a.eps_n = c->cfg.eta_l * a.inv_n;
    constexpr int TPB = multi_dn_threads<NB>();
    const dim3 grid((unsigned)c->chunks.size()), block(TPB);
    const bool any = a.refresh_mask != 0;
    Timer tm(c, HALOS_K_ARRIVE_MULTI, NB, 16 + 3 * c->wb * NB + (push ? 8 : 0) + (any ? 8 : 0));
    const Chunk* table = next_table(c);
    if (stats_on(c)) {
#define CALL(A, P) arrive_multi_dn_kernel<W, NB, A, P, true, kStream, kVE, TPB><<<grid, block, 0, c->stream>>>(table, a)
        HALOS_PICK2(any, push, CALL);
#undef CALL
    } else {
#define CALL(A, P) arrive_multi_dn_kernel<W, NB, A, P, false, kStream, kVE, TPB><<<grid, block, 0, c->stream>>>(table, a)
        HALOS_PICK2(any, push, CALL);
#undef CALL
    }
    tm.stop();
    c->launches++;
    c->batched_arrivals += NB;
    c->multi_launches++;
    CU(c, cudaGetLastError());
    return HALOS_OK;
}

template <class W, int NB>
int launch_arrive_multi(halos_ctx* c, LpsState& s, const Deferred* d, bool push) {
    if (c->cfg.optimizer == HALOS_OPT_DELAYED_NESTEROV) return launch_arrive_multi_dn<W, NB>(c, s, d, push);
    ArriveMultiArgs<W> a;
    const size_t nt = c->tensor_numel.size();
    for (int j = 0; j < kMaxBatch; ++j) {
        const int k = j < NB ? j : 0;
        a.h_flat[j] = (const W*)d[k].flat;
        a.h_ptrs[j] = d[k].flat ? nullptr : (const W* const*)(c->d_ptr_tables + (size_t)d[k].worker * nt);
        a.th0[j] = (W*)c->workers[d[k].worker].th0;
    }
    a.tensor_off = c->d_tensor_off;
    a.th = s.th;
    a.ml = s.ml;
    a.anchor = s.anchor;
    a.outbox = s.outbox;
    a.partial_delta = c->d_partial_delta;
    a.partial_theta = c->d_partial_theta;
    a.partial_Delta = c->d_partial_Delta;
    a.eta = c->cfg.eta_l;
    a.beta = c->cfg.beta_l;
    a.omb = 1.0f - c->cfg.beta_l;
    constexpr int TPB = multi_threads<NB>();
    const dim3 grid((unsigned)c->chunks.size()), block(TPB);
    Timer tm(c, HALOS_K_ARRIVE_MULTI, NB, 16 + 3 * c->wb * NB + (push ? 8 : 0));
    const Chunk* table = next_table(c);
#define CALL(P, S) arrive_multi_kernel<W, NB, P, S, kStream, kVE, TPB><<<grid, block, 0, c->stream>>>(table, a)
    HALOS_PICK2(push, stats_on(c), CALL);
#undef CALL
    tm.stop();
    c->launches++;
    c->batched_arrivals += NB;
    c->multi_launches++;
    CU(c, cudaGetLastError());
    return HALOS_OK;
}

template <class W>
int flush_deferred_t(halos_ctx* c, uint32_t lps, std::vector<Deferred>& q, bool push) {
    LpsState& s = c->lps[lps];
    if (q.empty()) return HALOS_OK;
    int rc = HALOS_OK;
    CU(c, cudaSetDevice(c->cfg.device));
    for (const Deferred& d : q)
        if ((rc = wait_fetch(c, c->workers[d.worker])) != HALOS_OK) return rc;
    switch (q.size()) {
        case 1: rc = launch_arrive<W>(c, s, c->workers[q[0].worker], q[0].worker, push, q[0].flat, q[0].refresh ? 1 : 0); break;
        case 2: rc = launch_arrive_multi<W, 2>(c, s, q.data(), push); break;
        case 3: rc = launch_arrive_multi<W, 3>(c, s, q.data(), push); break;
        case 4: rc = launch_arrive_multi<W, 4>(c, s, q.data(), push); break;
        case 5: rc = launch_arrive_multi<W, 5>(c, s, q.data(), push); break;
        case 6: rc = launch_arrive_multi<W, 6>(c, s, q.data(), push); break;
        case 7: rc = launch_arrive_multi<W, 7>(c, s, q.data(), push); break;
        case 8: rc = launch_arrive_multi<W, 8>(c, s, q.data(), push); break;
        default: rc = fail(c, HALOS_ERR_INVALID_ARG, "internal: batch larger than %d", kMaxBatch);
    }
    if (rc == HALOS_OK && stats_on(c)) {
        uint64_t seq[kMaxBatch];
        for (size_t j = 0; j < q.size(); ++j) seq[j] = q[j].seq;
        rc = finalize_stats(c, lps, (uint32_t)q.size(), push, seq);
    }
    q.clear();
    return rc;
}

int flush_deferred(halos_ctx* c, uint32_t lps, std::vector<Deferred>& q, bool push) {
    return c->wb == 4 ? flush_deferred_t<float>(c, lps, q, push) : flush_deferred_t<uint16_t>(c, lps, q, push);
}

// Launch everything that is still queued (a queued arrival never carries a push: those are flushed at once).
int flush_all(halos_ctx* c) {
    int rc = HALOS_OK;
    for (uint32_t l = 0; l < c->deferred.size(); ++l) {
        if (c->deferred[l].empty()) continue;
        int rf = flush_deferred(c, l, c->deferred[l], false);
        if (rc == HALOS_OK) rc = rf;
    }
    return rc;
}

// Launch what a reader of one state buffer depends on: the queue of that LPS, or of that worker's LPS if the
// worker has an arrival queued; the GPS buffers never wait (GPS events are not deferred).
int flush_worker(halos_ctx* c, uint32_t worker);
int flush_for(halos_ctx* c, uint32_t which, uint32_t index) {
    switch (which) {
        case HALOS_BUF_THETA_L: case HALOS_BUF_M_L: case HALOS_BUF_ANCHOR: case HALOS_BUF_OUTBOX: case HALOS_BUF_INBOX:
        case HALOS_BUF_ACC_L:
            if (index < c->deferred.size() && !c->deferred[index].empty()) return flush_deferred(c, index, c->deferred[index], false);
            return HALOS_OK;
        case HALOS_BUF_THETA0:
            return index < c->workers.size() ? flush_worker(c, index) : HALOS_OK;
        default:
            return HALOS_OK;
    }
}

// Before the pointer table or the result buffer of a worker is replaced, its queued arrival must have been launched.
int flush_worker(halos_ctx* c, uint32_t worker) {
    std::vector<Deferred>& q = c->deferred[c->workers[worker].lps];
    for (const Deferred& d : q)
        if (d.worker == worker) return flush_deferred(c, c->workers[worker].lps, q, false);
    return HALOS_OK;
}

}  // namespace

// ====================================================================================== C ABI
extern "C" {

void halos_default_config(halos_config* cfg) {
    if (!cfg) return;
    std::memset(cfg, 0, sizeof *cfg);
    cfg->struct_size = (uint32_t)sizeof(halos_config);
    cfg->eta_l = 0.2f;
    cfg->beta_l = 0.9f;
    cfg->eta_g = 0.15f;
    cfg->beta_g = 0.5f;
    cfg->alpha = 0.25f;
    cfg->K = 32;
    cfg->worker_dtype = HALOS_F32;
    cfg->optimizer = HALOS_OPT_PAPER;
    cfg->delay_l = 1;
    cfg->delay_g = 1;
}

int halos_create(const halos_config* cfg, const float* theta_init_dev, halos_ctx** out) {
    if (!cfg || !out || !theta_init_dev) return fail(nullptr, HALOS_ERR_INVALID_ARG, "null argument");
    if (cfg->struct_size != sizeof(halos_config)) return fail(nullptr, HALOS_ERR_INVALID_ARG, "struct_size mismatch");
    if (cfg->n_lps == 0 || cfg->n_workers == 0 || cfg->n_tensors == 0 || !cfg->worker_lps || !cfg->tensor_numel)
        return fail(nullptr, HALOS_ERR_INVALID_ARG, "empty configuration");
    if (cfg->n_lps > 255 || cfg->n_workers > 65535) return fail(nullptr, HALOS_ERR_INVALID_ARG, "too many servers or workers");
    if (cfg->K == 0) return fail(nullptr, HALOS_ERR_INVALID_ARG, "K must be positive");
    if (cfg->worker_dtype != HALOS_F32 && cfg->worker_dtype != HALOS_BF16)
        return fail(nullptr, HALOS_ERR_INVALID_ARG, "unknown worker_dtype");
    if (cfg->optimizer != HALOS_OPT_PAPER && cfg->optimizer != HALOS_OPT_DELAYED_NESTEROV)
        return fail(nullptr, HALOS_ERR_INVALID_ARG, "unknown optimizer");
    if (cfg->optimizer == HALOS_OPT_DELAYED_NESTEROV && (cfg->delay_l == 0 || cfg->delay_g == 0))
        return fail(nullptr, HALOS_ERR_INVALID_ARG, "delays must be at least 1");
    if ((cfg->flags & HALOS_FLAG_MATERIALISE_DELTA) && cfg->optimizer == HALOS_OPT_DELAYED_NESTEROV)
        return fail(nullptr, HALOS_ERR_UNSUPPORTED, "materialised deltas do not combine with delayed Nesterov");
    if ((cfg->alloc == nullptr) != (cfg->free_ == nullptr)) return fail(nullptr, HALOS_ERR_INVALID_ARG, "alloc and free_ go together");
    for (uint32_t w = 0; w < cfg->n_workers; ++w)
        if (cfg->worker_lps[w] >= cfg->n_lps) return fail(nullptr, HALOS_ERR_INVALID_ARG, "worker_lps[%u] out of range", w);
    uint32_t chunk_elems = cfg->chunk_elems ? cfg->chunk_elems : kDefaultChunkElems;
    if (chunk_elems % 8 != 0) return fail(nullptr, HALOS_ERR_INVALID_ARG, "chunk_elems must be a positive multiple of 8");
    if ((cfg->flags & HALOS_FLAG_STATS) && chunk_elems > kStatMaxChunk)
        return fail(nullptr, HALOS_ERR_UNSUPPORTED, "statistics need chunk_elems <= %u", kStatMaxChunk);

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
        (void)cudaGetLastError();
        return fail(nullptr, HALOS_ERR_CUDA, "no CUDA device: this library has no CPU path");
    }
    if (cfg->device < 0 || cfg->device >= ndev) return fail(nullptr, HALOS_ERR_INVALID_ARG, "device ordinal out of range");

    halos_ctx* c = new (std::nothrow) halos_ctx();
    if (!c) return fail(nullptr, HALOS_ERR_OOM, "host allocation failed");
    c->cfg = *cfg;
    c->cfg.worker_lps = nullptr;
    c->cfg.tensor_numel = nullptr;
    c->stream = (cudaStream_t)cfg->stream;
    c->wb = cfg->worker_dtype == HALOS_F32 ? 4 : 2;
    c->worker_lps.assign(cfg->worker_lps, cfg->worker_lps + cfg->n_workers);
    c->tensor_numel.assign(cfg->tensor_numel, cfg->tensor_numel + cfg->n_tensors);
    c->tensor_off.resize(cfg->n_tensors + 1);
    c->tensor_off[0] = 0;
    for (uint32_t k = 0; k < cfg->n_tensors; ++k) c->tensor_off[k + 1] = c->tensor_off[k] + c->tensor_numel[k];
    c->P = c->tensor_off[cfg->n_tensors];
    if (c->P == 0) {
        delete c;
        return fail(nullptr, HALOS_ERR_INVALID_ARG, "P = 0");
    }
    build_chunks(c, chunk_elems);

    auto bail = [&](int status, const char* what) {
        std::string msg = c->err.empty() ? what : c->err;
        release(c);
        delete c;
        return fail(nullptr, status, "%s", msg.c_str());
    };
#define CUC(call)                                                                  \
    do {                                                                           \
        cudaError_t e_ = (call);                                                   \
        if (e_ != cudaSuccess) {                                                   \
            c->err = std::string(#call) + ": " + cudaGetErrorString(e_);           \
            return bail(HALOS_ERR_CUDA, "cuda");                                   \
        }                                                                          \
    } while (0)

    CUC(cudaSetDevice(cfg->device));
    const size_t P = c->P, nt = cfg->n_tensors, nc = c->chunks.size();
    auto A = [&](size_t bytes) { return dev_alloc(c, bytes); };
    // State buffers: with HALOS_FLAG_GUARD each gets a 256-byte canary zone on both sides.
    const bool guard = (cfg->flags & HALOS_FLAG_GUARD) != 0;
    auto S = [&](size_t bytes) -> void* {
        if (!guard) return dev_alloc(c, bytes);
        const size_t padded = (bytes + 255) / 256 * 256;
        char* raw = (char*)dev_alloc(c, padded + 2 * kGuardBytes);
        if (!raw) return nullptr;
        c->guards.push_back(GuardedBuffer{raw, padded, bytes});
        return raw + kGuardBytes;
    };
    bool ok = true;
    ok &= (c->d_chunks = (Chunk*)A(nc * sizeof(Chunk))) != nullptr;
    ok &= (c->d_chunks_rev = (Chunk*)A(nc * sizeof(Chunk))) != nullptr;
    ok &= (c->d_tensor_off = (unsigned long long*)A((nt + 1) * 8)) != nullptr;
    ok &= (c->d_tensor_chunk_begin = (uint32_t*)A((nt + 1) * 4)) != nullptr;
    ok &= (c->d_ptr_tables = (const void**)A((size_t)cfg->n_workers * nt * 8)) != nullptr;
    if (cfg->flags & HALOS_FLAG_STATS) {
        ok &= (c->d_partial_delta = (double*)A((size_t)kMaxBatch * nc * 8)) != nullptr;   // [arrival of a launch][chunk]
        ok &= (c->d_partial_Delta = (double*)A(nc * 8)) != nullptr;
        ok &= (c->d_partial_theta = (double*)A((size_t)kMaxBatch * nc * 8)) != nullptr;
        ok &= (c->d_stats = (double*)A((size_t)3 * cfg->n_lps * nt * 8)) != nullptr;
    }
    ok &= (c->Theta = (float*)S(P * 4)) != nullptr;
    ok &= (c->Mg = (float*)S(P * 4)) != nullptr;
    const bool dn = cfg->optimizer == HALOS_OPT_DELAYED_NESTEROV;
    if (dn) ok &= (c->acc_g = (float*)S(P * 4)) != nullptr;
    c->lps.resize(cfg->n_lps);
    c->deferred.resize(cfg->n_lps);
    for (auto& s : c->lps) {
        if (!ok) break;
        ok &= (s.th = (float*)S(P * 4)) != nullptr;
        ok &= (s.ml = (float*)S(P * 4)) != nullptr;
        ok &= (s.anchor = (float*)S(P * 4)) != nullptr;
        ok &= (s.outbox = (float*)S(P * 4)) != nullptr;
        ok &= (s.inbox = (float*)S(P * 4)) != nullptr;
        if (dn) ok &= (s.acc = (float*)S(P * 4)) != nullptr;
    }
    c->workers.resize(cfg->n_workers);
    for (uint32_t w = 0; w < cfg->n_workers && ok; ++w) {
        c->workers[w].lps = c->worker_lps[w];
        ok &= (c->workers[w].th0 = S(P * c->wb)) != nullptr;
        if (ok && (cfg->flags & HALOS_FLAG_MATERIALISE_DELTA)) ok &= (c->workers[w].delta = (float*)S(P * 4)) != nullptr;
    }
    if (!ok) return bail(HALOS_ERR_OOM, "device allocation failed");
    for (auto& g : c->guards) {   // canaries: 0xA5 before the data, and from the end of the data to the end of the block
        CUC(cudaMemsetAsync(g.raw, 0xA5, kGuardBytes, c->stream));
        CUC(cudaMemsetAsync(g.raw + kGuardBytes + g.bytes, 0xA5, g.padded - g.bytes + kGuardBytes, c->stream));
    }
    for (void* p : c->owned)
        if (reinterpret_cast<uintptr_t>(p) & 255) return bail(HALOS_ERR_INVALID_ARG, "allocator returned a pointer not aligned to 256 bytes");

    CUC(cudaHostAlloc((void**)&c->h_ptr_tables, (size_t)cfg->n_workers * nt * 8, cudaHostAllocDefault));
    for (auto& w : c->workers) CUC(cudaEventCreateWithFlags(&w.table_copied, cudaEventDisableTiming));
    CUC(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
    for (int s = 0; s < kStageSlots; ++s) {
        CUC(cudaEventCreateWithFlags(&c->stage_ready[s], cudaEventDisableTiming));
        CUC(cudaEventCreateWithFlags(&c->stage_free[s], cudaEventDisableTiming));
    }

    cudaStream_t st = c->stream;
    CUC(cudaMemcpyAsync(c->d_chunks, c->chunks.data(), nc * sizeof(Chunk), cudaMemcpyHostToDevice, st));
    std::vector<Chunk> reversed(c->chunks.rbegin(), c->chunks.rend());
    CUC(cudaMemcpyAsync(c->d_chunks_rev, reversed.data(), nc * sizeof(Chunk), cudaMemcpyHostToDevice, st));
    CUC(cudaMemcpyAsync(c->d_tensor_off, c->tensor_off.data(), (nt + 1) * 8, cudaMemcpyHostToDevice, st));
    CUC(cudaMemcpyAsync(c->d_tensor_chunk_begin, c->tensor_chunk_begin.data(), (nt + 1) * 4, cudaMemcpyHostToDevice, st));
    if (c->d_stats) CUC(cudaMemsetAsync(c->d_stats, 0, (size_t)3 * cfg->n_lps * nt * 8, st));
    // Alg. 1 lines 6-7
    CUC(cudaMemcpyAsync(c->Theta, theta_init_dev, P * 4, cudaMemcpyDeviceToDevice, st));
    CUC(cudaMemsetAsync(c->Mg, 0, P * 4, st));
    if (c->acc_g) CUC(cudaMemsetAsync(c->acc_g, 0, P * 4, st));
    for (auto& s : c->lps) {
        CUC(cudaMemcpyAsync(s.th, theta_init_dev, P * 4, cudaMemcpyDeviceToDevice, st));
        CUC(cudaMemcpyAsync(s.anchor, theta_init_dev, P * 4, cudaMemcpyDeviceToDevice, st));
        CUC(cudaMemsetAsync(s.ml, 0, P * 4, st));
        CUC(cudaMemsetAsync(s.outbox, 0, P * 4, st));
        CUC(cudaMemsetAsync(s.inbox, 0, P * 4, st));
        if (s.acc) CUC(cudaMemsetAsync(s.acc, 0, P * 4, st));
    }
    for (auto& w : c->workers) {
        if (c->wb == 4) {
            CUC(cudaMemcpyAsync(w.th0, theta_init_dev, P * 4, cudaMemcpyDeviceToDevice, st));
        } else {
            cast_bf16_kernel<<<1184, 256, 0, st>>>(theta_init_dev, (uint16_t*)w.th0, (unsigned long long)P);
            CUC(cudaGetLastError());
        }
    }
    CUC(cudaStreamSynchronize(st));
#undef CUC
    *out = c;
    return HALOS_OK;
}

int halos_destroy(halos_ctx* c) {
    if (!c) return HALOS_OK;
    cudaSetDevice(c->cfg.device);
    (void)flush_all(c);
    release(c);
    delete c;
    return HALOS_OK;
}

int halos_worker_delta(halos_ctx* c, uint32_t worker, const void* flat, const void* const* ptrs) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (worker >= c->cfg.n_workers) return fail(c, HALOS_ERR_INVALID_ARG, "worker out of range");
    if ((flat == nullptr) == (ptrs == nullptr)) return fail(c, HALOS_ERR_INVALID_ARG, "give exactly one of flat / pointer table");
    WorkerState& w = c->workers[worker];
    if (w.pending != PEND_NONE) return fail(c, HALOS_ERR_BAD_STATE, "worker %u already has a pending result", worker);
    {
        int rq = flush_worker(c, worker);   // a still-queued arrival of this worker reads its old result / table
        if (rq != HALOS_OK) return rq;
    }
    if (stats_on(c)) {
        // which tensors of this result can take the vector path (their first full chunk starts `head` elements in)
        const size_t ntens = c->tensor_numel.size();
        w.vec_aligned.assign(ntens, 0);
        for (size_t k = 0; k < ntens; ++k) {
            const uint64_t head = (kVE - (c->tensor_off[k] % kVE)) % kVE;
            const uintptr_t first = flat ? reinterpret_cast<uintptr_t>(flat) + (c->tensor_off[k] + head) * c->wb
                                         : reinterpret_cast<uintptr_t>(ptrs[k]) + head * c->wb;
            w.vec_aligned[k] = (first % (kVE * c->wb)) == 0;
        }
    }
    if (flat) {
        if (reinterpret_cast<uintptr_t>(flat) % c->wb) return fail(c, HALOS_ERR_INVALID_ARG, "thetaH not aligned to its element size");
        if (c->cfg.flags & HALOS_FLAG_MATERIALISE_DELTA) {
            CU(c, cudaSetDevice(c->cfg.device));
            int rc = launch_delta(c, worker, flat);
            if (rc != HALOS_OK) return rc;
            w.pending = PEND_DELTA;
            return HALOS_OK;
        }
        w.flat = flat;
        w.pending = PEND_FLAT;
        return HALOS_OK;
    }
    const size_t nt = c->tensor_numel.size();
    for (size_t k = 0; k < nt; ++k) {
        if (!ptrs[k] && c->tensor_numel[k]) return fail(c, HALOS_ERR_INVALID_ARG, "null pointer for tensor %zu", k);
        if (reinterpret_cast<uintptr_t>(ptrs[k]) % c->wb) return fail(c, HALOS_ERR_INVALID_ARG, "tensor %zu not aligned to its element size", k);
    }
    CU(c, cudaSetDevice(c->cfg.device));
    CU(c, cudaEventSynchronize(w.table_copied));  // the previous upload from this pinned slot has left the host
    const void** slot = c->h_ptr_tables + (size_t)worker * nt;
    std::memcpy(slot, ptrs, nt * 8);
    CU(c, cudaMemcpyAsync(c->d_ptr_tables + (size_t)worker * nt, slot, nt * 8, cudaMemcpyHostToDevice, c->stream));
    CU(c, cudaEventRecord(w.table_copied, c->stream));
    if (c->cfg.flags & HALOS_FLAG_MATERIALISE_DELTA) {
        int rc = launch_delta(c, worker, nullptr);
        if (rc != HALOS_OK) return rc;
        w.pending = PEND_DELTA;
        return HALOS_OK;
    }
    w.pending = PEND_PTRS;
    return HALOS_OK;
}

int halos_worker_delta_host(halos_ctx* c, uint32_t worker, const void* host) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (worker >= c->cfg.n_workers || !host) return fail(c, HALOS_ERR_INVALID_ARG, "bad worker or null pointer");
    WorkerState& w = c->workers[worker];
    if (w.pending != PEND_NONE) return fail(c, HALOS_ERR_BAD_STATE, "worker %u already has a pending result", worker);
    {
        int rq = flush_worker(c, worker);
        if (rq != HALOS_OK) return rq;
    }
    int slot = -1;
    for (int k = 0; k < kStageSlots; ++k) {
        int s = (c->stage_next + k) % kStageSlots;
        if (c->stage_owner[s] < 0) {
            slot = s;
            break;
        }
    }
    if (slot < 0) return fail(c, HALOS_ERR_BAD_STATE, "all %d staging buffers hold results that were not applied yet", kStageSlots);
    CU(c, cudaSetDevice(c->cfg.device));
    if (!c->stage[slot]) {
        c->stage[slot] = dev_alloc(c, c->P * c->wb);
        if (!c->stage[slot]) return fail(c, HALOS_ERR_OOM, "staging buffer allocation failed");
    }
    // The copy runs on the context's own copy stream so that it overlaps the update kernels of
    // earlier events; stage_free orders it after the kernel that last read this slot.
    CU(c, cudaStreamWaitEvent(c->copy_stream, c->stage_free[slot], 0));
    CU(c, cudaMemcpyAsync(c->stage[slot], host, c->P * c->wb, cudaMemcpyHostToDevice, c->copy_stream));
    CU(c, cudaEventRecord(c->stage_ready[slot], c->copy_stream));
    if (c->cfg.flags & HALOS_FLAG_MATERIALISE_DELTA) {
        // delta is formed as soon as the copy has landed and the staging buffer is free again at once
        CU(c, cudaStreamWaitEvent(c->stream, c->stage_ready[slot], 0));
        int rc = launch_delta(c, worker, c->stage[slot]);
        if (rc != HALOS_OK) return rc;
        CU(c, cudaEventRecord(c->stage_free[slot], c->stream));
        c->stage_next = (slot + 1) % kStageSlots;
        w.pending = PEND_DELTA;
        return HALOS_OK;
    }
    c->stage_owner[slot] = (int)worker;
    c->stage_next = (slot + 1) % kStageSlots;
    w.slot = slot;
    w.pending = PEND_STAGED;
    return HALOS_OK;
}

int halos_worker_fetch_host(halos_ctx* c, uint32_t worker, void* dst_host) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (worker >= c->cfg.n_workers || !dst_host) return fail(c, HALOS_ERR_INVALID_ARG, "bad worker or null pointer");
    {
        int rq = flush_worker(c, worker);   // the snapshot is written by this worker's arrival, which may still be queued
        if (rq != HALOS_OK) return rq;
    }
    WorkerState& w = c->workers[worker];
    CU(c, cudaSetDevice(c->cfg.device));
    if (!c->d2h_stream) CU(c, cudaStreamCreateWithFlags(&c->d2h_stream, cudaStreamNonBlocking));
    if (!w.snap_ready) CU(c, cudaEventCreateWithFlags(&w.snap_ready, cudaEventDisableTiming));
    if (!w.fetched) CU(c, cudaEventCreateWithFlags(&w.fetched, cudaEventDisableTiming));
    CU(c, cudaEventRecord(w.snap_ready, c->stream));
    CU(c, cudaStreamWaitEvent(c->d2h_stream, w.snap_ready, 0));
    CU(c, cudaMemcpyAsync(dst_host, w.th0, c->P * c->wb, cudaMemcpyDeviceToHost, c->d2h_stream));
    CU(c, cudaEventRecord(w.fetched, c->d2h_stream));
    w.fetch_outstanding = true;
    return HALOS_OK;
}

int halos_fetch_sync(halos_ctx* c) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (!c->d2h_stream) return HALOS_OK;
    CU(c, cudaSetDevice(c->cfg.device));
    CU(c, cudaStreamSynchronize(c->d2h_stream));
    return HALOS_OK;
}

int halos_lps_apply(halos_ctx* c, uint32_t lps, uint32_t worker, int* push_due) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    int rq = flush_all(c);
    if (rq != HALOS_OK) return rq;
    return apply_impl(c, lps, worker, false, push_due);
}

int halos_lps_push(halos_ctx* c, uint32_t lps) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (lps >= c->cfg.n_lps) return fail(c, HALOS_ERR_INVALID_ARG, "lps out of range");
    {
        int rq = flush_all(c);
        if (rq != HALOS_OK) return rq;
    }
    LpsState& s = c->lps[lps];
    if (s.phase != HALOS_IDLE) return fail(c, HALOS_ERR_BAD_STATE, "LPS %u already has a round trip in flight", lps);
    CU(c, cudaSetDevice(c->cfg.device));
    PushArgs a{s.th, s.anchor, s.outbox, c->d_partial_Delta};
    const dim3 grid((unsigned)c->chunks.size()), block(kThreads);
    const bool stats = (c->cfg.flags & HALOS_FLAG_STATS) != 0;
    Timer tm(c, HALOS_K_PUSH, 0, 12);
    if (stats) push_kernel<true, kUnroll, kStream, kVE><<<grid, block, 0, c->stream>>>(next_table(c), a);
    else push_kernel<false, kUnroll, kStream, kVE><<<grid, block, 0, c->stream>>>(next_table(c), a);
    tm.stop();
    c->launches++;
    CU(c, cudaGetLastError());
    if (stats) {
        const uint32_t nt = (uint32_t)c->tensor_numel.size();
        stats_finalize_push_kernel<<<nt, 32, 0, c->stream>>>(c->d_partial_Delta, c->d_tensor_chunk_begin,
                                                             c->d_stats + ((size_t)1 * c->cfg.n_lps + lps) * nt, nt);
        c->launches++;
        CU(c, cudaGetLastError());
    }
    s.phase = HALOS_PUSHED;
    s.t_push = s.t;
    return HALOS_OK;
}

int halos_gps_merge(halos_ctx* c, uint32_t lps) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (lps >= c->cfg.n_lps) return fail(c, HALOS_ERR_INVALID_ARG, "lps out of range");
    LpsState& s = c->lps[lps];
    if (s.phase != HALOS_PUSHED) return fail(c, HALOS_ERR_BAD_STATE, "LPS %u has no Delta in flight", lps);
    CU(c, cudaSetDevice(c->cfg.device));
    const dim3 grid((unsigned)c->chunks.size()), block(kThreads);
    const bool gps_refresh = c->cfg.optimizer == HALOS_OPT_DELAYED_NESTEROV && ((c->gps_iter + 1) % c->cfg.delay_g) == 0;
    Timer tm(c, HALOS_K_GPS, 1, 24 + (gps_refresh ? 8 : 0));
    if (c->cfg.optimizer == HALOS_OPT_DELAYED_NESTEROV) {
        const float inv_n = 1.0f / (float)c->cfg.delay_g;
        GpsDnArgs a{s.outbox, c->Theta, c->Mg, c->acc_g, s.inbox, c->cfg.eta_g, c->cfg.beta_g, inv_n, c->cfg.eta_g * inv_n};
        if (((c->gps_iter + 1) % c->cfg.delay_g) == 0) gps_dn_kernel<true, kStream, kVE><<<grid, block, 0, c->stream>>>(next_table(c), a);
        else gps_dn_kernel<false, kStream, kVE><<<grid, block, 0, c->stream>>>(next_table(c), a);
    } else {
        GpsArgs a{s.outbox, c->Theta, c->Mg, s.inbox, c->cfg.eta_g, c->cfg.beta_g, 1.0f - c->cfg.beta_g};
        gps_kernel<kUnroll, kStream, kVE><<<grid, block, 0, c->stream>>>(next_table(c), a);
    }
    tm.stop();
    c->launches++;
    CU(c, cudaGetLastError());
    c->gps_iter += 1;
    s.inbox_iter = c->gps_iter;
    s.phase = HALOS_ANSWERED;
    return HALOS_OK;
}

static int pull_impl(halos_ctx* c, uint32_t lps);

int halos_lps_pull(halos_ctx* c, uint32_t lps) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    int rq = flush_all(c);
    if (rq != HALOS_OK) return rq;
    return pull_impl(c, lps);
}

// the caller has launched whatever was queued for this LPS
static int pull_impl(halos_ctx* c, uint32_t lps) {
    if (lps >= c->cfg.n_lps) return fail(c, HALOS_ERR_INVALID_ARG, "lps out of range");
    LpsState& s = c->lps[lps];
    if (s.phase != HALOS_ANSWERED) return fail(c, HALOS_ERR_BAD_STATE, "LPS %u has no Theta_i to merge", lps);
    CU(c, cudaSetDevice(c->cfg.device));
    PullArgs a{s.th, s.inbox, s.anchor, c->cfg.alpha, 1.0f - c->cfg.alpha};
    const dim3 grid((unsigned)c->chunks.size()), block(kThreads);
    Timer tm(c, HALOS_K_PULL, 1, 16);
    pull_kernel<kUnroll, kStream, kVE><<<grid, block, 0, c->stream>>>(next_table(c), a);
    tm.stop();
    c->launches++;
    CU(c, cudaGetLastError());
    s.t_last = s.t;
    s.phase = HALOS_IDLE;
    return HALOS_OK;
}

// GPS update for this LPS's Delta and the merge of the answer into the same LPS as one launch.  The caller has
// launched whatever was queued for this LPS.
static int gps_pull_impl(halos_ctx* c, uint32_t lps) {
    if (lps >= c->cfg.n_lps) return fail(c, HALOS_ERR_INVALID_ARG, "lps out of range");
    LpsState& s = c->lps[lps];
    if (s.phase != HALOS_PUSHED) return fail(c, HALOS_ERR_BAD_STATE, "LPS %u has no Delta in flight", lps);
    CU(c, cudaSetDevice(c->cfg.device));
    GpsPullArgs a;
    a.outbox = s.outbox;
    a.Theta = c->Theta;
    a.Mg = c->Mg;
    a.acc = c->acc_g;
    a.inbox = s.inbox;
    a.th = s.th;
    a.anchor = s.anchor;
    a.eta = c->cfg.eta_g;
    a.beta = c->cfg.beta_g;
    a.omb = 1.0f - c->cfg.beta_g;
    a.inv_n = 1.0f / (float)(c->cfg.delay_g ? c->cfg.delay_g : 1);
    a.eps_n = c->cfg.eta_g * a.inv_n;
    a.alpha = c->cfg.alpha;
    a.oma = 1.0f - c->cfg.alpha;
    const dim3 grid((unsigned)c->chunks.size()), block(kThreads);
    const bool gps_refresh = c->cfg.optimizer == HALOS_OPT_DELAYED_NESTEROV && ((c->gps_iter + 1) % c->cfg.delay_g) == 0;
    Timer tm(c, HALOS_K_GPS_PULL, 2, 36 + (gps_refresh ? 8 : 0));
    const Chunk* table = next_table(c);
    if (c->cfg.optimizer != HALOS_OPT_DELAYED_NESTEROV) gps_pull_kernel<0, kStream, kVE><<<grid, block, 0, c->stream>>>(table, a);
    else if (((c->gps_iter + 1) % c->cfg.delay_g) == 0) gps_pull_kernel<2, kStream, kVE><<<grid, block, 0, c->stream>>>(table, a);
    else gps_pull_kernel<1, kStream, kVE><<<grid, block, 0, c->stream>>>(table, a);
    tm.stop();
    c->launches++;
    CU(c, cudaGetLastError());
    c->gps_iter += 1;
    s.inbox_iter = c->gps_iter;
    s.t_last = s.t;
    s.phase = HALOS_IDLE;
    return HALOS_OK;
}

int halos_gps_merge_pull(halos_ctx* c, uint32_t lps) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    int rq = flush_all(c);
    if (rq != HALOS_OK) return rq;
    return gps_pull_impl(c, lps);
}

// ------------------------------------------------------------------------------ event-queue driver
// Events are taken in trace order: counters, phases, the log and the producer calls follow that order
// exactly.  With max_batch > 1 the LAUNCH of an arrival may be deferred: arrivals at one LPS wait in
// that LPS's queue and are flushed as one multi-arrival launch when the queue is full, when the same
// worker arrives again, when the arrival closes a window of K (it is flushed with the push fused), when
// a PULL for that LPS comes up, or at the end.  Everything an arrival at LPS l touches (theta_l, m_l,
// the worker's snapshot; outbox_l only when it pushes) is disjoint from what events of other LPSs and
// GPS_RECV(l) touch, so the deferred launches commute with the launches they are moved past and the
// final state is bit-identical to the unbatched replay.
int halos_replay_stream(halos_ctx* c, const halos_event* ev, uint32_t n, halos_producer_fn producer, void* user,
                        halos_event_log* log, uint32_t* failed_at, uint32_t max_batch) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (n && !ev) return fail(c, HALOS_ERR_INVALID_ARG, "null event array");
    if (max_batch == 0) max_batch = 1;
    if (max_batch > (uint32_t)kMaxBatch) max_batch = kMaxBatch;
    const bool immediate = (c->cfg.flags & HALOS_FLAG_MATERIALISE_DELTA) != 0;   // launched event by event
    std::vector<std::vector<Deferred>>& queue = c->deferred;
    int rc = HALOS_OK;
    uint32_t k = 0;
    for (; k < n && rc == HALOS_OK; ++k) {
        const halos_event& e = ev[k];
        halos_event_log rec;
        std::memset(&rec, 0, sizeof rec);
        rec.index = k;
        rec.kind = e.kind;
        rec.lps = e.lps;
        rec.worker = e.worker;
        if (e.lps >= c->cfg.n_lps) rc = fail(c, HALOS_ERR_INVALID_ARG, "event %u: lps out of range", k);
        else if (e.kind == HALOS_EV_ARRIVE) {
            std::vector<Deferred>& q = queue[e.lps];
            if (e.worker >= c->cfg.n_workers) rc = fail(c, HALOS_ERR_INVALID_ARG, "event %u: worker out of range", k);
            else if (!producer && c->workers[e.worker].pending == PEND_NONE) rc = fail(c, HALOS_ERR_INVALID_ARG, "ARRIVE events need a producer");
            else {
                WorkerState& w = c->workers[e.worker];
                for (const Deferred& d : q)
                    if (d.worker == e.worker) {   // its previous result is still queued: run it first
                        rc = flush_deferred(c, e.lps, q, false);
                        break;
                    }
                const void* flat = nullptr;
                const void* const* ptrs = nullptr;
                bool due = false, push = false;
                // membership and the state of the round trip are checked before the producer is asked, so
                // that a refused event registers nothing
                if (rc == HALOS_OK) rc = arrival_check(c, e.lps, e.worker, true, &due, &push);
                if (rc == HALOS_OK && w.pending == PEND_NONE) {
                    if (producer(user, k, e.worker, w.round, &flat, &ptrs) != 0)
                        rc = fail(c, HALOS_ERR_INVALID_ARG, "event %u: producer failed", k);
                    else rc = halos_worker_delta(c, e.worker, flat, ptrs);
                }
                if (rc == HALOS_OK && (w.pending == PEND_STAGED || immediate) && !q.empty()) rc = flush_deferred(c, e.lps, q, false);
                if (rc == HALOS_OK) {
                    rec.worker_staleness = c->lps[e.lps].t - w.sched_t;
                    if (w.pending == PEND_STAGED || immediate) {
                        rc = apply_impl(c, e.lps, e.worker, true, nullptr);   // host-staged results are not deferred
                    } else {
                        const bool refresh = c->cfg.optimizer == HALOS_OPT_DELAYED_NESTEROV &&
                                             ((c->lps[e.lps].t + 1) % c->cfg.delay_l) == 0;
                        // statistics are reduced per vector or per element depending on the alignment of the
                        // caller's tensors; only arrivals that agree on it tensor by tensor share a launch, so that
                        // a fused launch reports the sums of the single launches bit for bit
                        if (stats_on(c) && !q.empty() && c->workers[q[0].worker].vec_aligned != w.vec_aligned)
                            rc = flush_deferred(c, e.lps, q, false);
                        if (rc == HALOS_OK) {
                            q.push_back(Deferred{e.worker, w.pending == PEND_FLAT ? w.flat : nullptr, refresh, c->stats_seq++});
                            rec.fused = (uint8_t)(q.size() > 1 || push);
                            apply_commit(c, e.lps, e.worker, push);
                            if (push || q.size() >= max_batch) rc = flush_deferred(c, e.lps, q, push);
                        }
                    }
                    rec.pushed = (uint8_t)push;
                }
            }
        } else if (e.kind == HALOS_EV_GPS_RECV) {
            // GPS_RECV(l) directly followed by PULL(l): one fused launch (only with multi-event fusion enabled)
            if (max_batch > 1 && k + 1 < n && ev[k + 1].kind == HALOS_EV_PULL && ev[k + 1].lps == e.lps &&
                c->lps[e.lps].phase == HALOS_PUSHED) {
                rc = flush_deferred(c, e.lps, queue[e.lps], false);   // arrivals before the PULL come first
                const uint64_t t_last_before = c->lps[e.lps].t_last;
                if (rc == HALOS_OK) rc = gps_pull_impl(c, e.lps);
                if (rc == HALOS_OK) {
                    rec.fused = 1;
                    if (log) {
                        rec.t = c->lps[e.lps].t;
                        rec.t_last = t_last_before;
                        rec.gps_iter = c->gps_iter;
                        log[k] = rec;
                    }
                    ++k;                                              // the PULL is done as well
                    std::memset(&rec, 0, sizeof rec);
                    rec.index = k;
                    rec.kind = HALOS_EV_PULL;
                    rec.lps = e.lps;
                    rec.fused = 1;
                    rec.gps_lag = 0;                                  // it merges the Theta_i this very iteration produced
                }
            } else {
                rc = halos_gps_merge(c, e.lps);
            }
        } else if (e.kind == HALOS_EV_PULL) {
            rc = flush_deferred(c, e.lps, queue[e.lps], false);
            if (rc == HALOS_OK) {
                if (c->lps[e.lps].phase == HALOS_ANSWERED) rec.gps_lag = c->gps_iter - c->lps[e.lps].inbox_iter;
                rc = pull_impl(c, e.lps);
            }
        } else {
            rc = fail(c, HALOS_ERR_INVALID_ARG, "event %u: unknown kind %u", k, (unsigned)e.kind);
        }
        if (rc == HALOS_OK && log) {
            rec.t = c->lps[e.lps].t;
            rec.t_last = c->lps[e.lps].t_last;
            rec.gps_iter = c->gps_iter;
            log[k] = rec;
        }
    }
    if (rc != HALOS_OK) {
        (void)flush_all(c);   // events before the failing one stay applied: launch what they queued
        if (failed_at) *failed_at = k ? k - 1 : 0;
    }
    return rc;
}

int halos_flush(halos_ctx* c) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    return flush_all(c);
}

int halos_replay_batched(halos_ctx* c, const halos_event* ev, uint32_t n, halos_producer_fn producer, void* user,
                         halos_event_log* log, uint32_t* failed_at, uint32_t max_batch) {
    int rc = halos_replay_stream(c, ev, n, producer, user, log, failed_at, max_batch);
    if (!c) return rc;
    int rf = flush_all(c);   // whatever is still queued belongs to events already accounted for
    return rc != HALOS_OK ? rc : rf;
}

// Producer over a table of results: entry k is the flat result of event k (ARRIVE events only).
static int table_producer(void* user, uint32_t event_index, uint32_t, uint64_t, const void** flat_dev, const void* const**) {
    *flat_dev = static_cast<const void* const*>(user)[event_index];
    return *flat_dev ? 0 : 1;
}

int halos_replay_results(halos_ctx* c, const halos_event* ev, uint32_t n, const void* const* results_host, halos_event_log* log,
                         uint32_t* failed_at, uint32_t max_batch, int keep_queued) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (n && !results_host) return fail(c, HALOS_ERR_INVALID_ARG, "null result table");
    void* user = const_cast<void*>(static_cast<const void*>(results_host));
    return keep_queued ? halos_replay_stream(c, ev, n, table_producer, user, log, failed_at, max_batch)
                       : halos_replay_batched(c, ev, n, table_producer, user, log, failed_at, max_batch);
}

int halos_replay(halos_ctx* c, const halos_event* ev, uint32_t n, halos_producer_fn producer, void* user,
                 halos_event_log* log, uint32_t* failed_at) {
    return halos_replay_batched(c, ev, n, producer, user, log, failed_at, 1);
}

// ------------------------------------------------------------------------------ checkpoint / resume
namespace {
struct CkptHeader {
    char magic[8];
    uint32_t version, wb;
    uint64_t P;
    uint32_t n_lps, n_workers, n_tensors, K;
    float eta_l, beta_l, eta_g, beta_g, alpha;
    uint32_t optimizer;
    uint64_t gps_iter;
    uint32_t delay_l, delay_g;
};
struct CkptLps { uint64_t t, t_last, t_push, inbox_iter; int32_t phase; int32_t pad; };
struct CkptWorker { uint64_t round, sched_t; };
constexpr size_t kBounce = 64u << 20;

int stream_buffer(halos_ctx* c, FILE* f, void* dev, size_t bytes, bool to_file, void* bounce) {
    for (size_t off = 0; off < bytes; off += kBounce) {
        const size_t n = bytes - off < kBounce ? bytes - off : kBounce;
        if (to_file) {
            CU(c, cudaMemcpyAsync(bounce, (char*)dev + off, n, cudaMemcpyDeviceToHost, c->stream));
            CU(c, cudaStreamSynchronize(c->stream));
            if (fwrite(bounce, 1, n, f) != n) return fail(c, HALOS_ERR_INVALID_ARG, "short write to checkpoint file");
        } else {
            if (fread(bounce, 1, n, f) != n) return fail(c, HALOS_ERR_INVALID_ARG, "checkpoint file is truncated");
            CU(c, cudaMemcpyAsync((char*)dev + off, bounce, n, cudaMemcpyHostToDevice, c->stream));
            CU(c, cudaStreamSynchronize(c->stream));
        }
    }
    return HALOS_OK;
}

int checkpoint(halos_ctx* c, const char* path, bool to_file) {
    if (!c || !path) return HALOS_ERR_INVALID_ARG;
    {
        int rq = flush_all(c);
        if (rq != HALOS_OK) return rq;
    }
    for (auto& w : c->workers)
        if (w.pending != PEND_NONE) return fail(c, HALOS_ERR_BAD_STATE, "a worker result is registered but not applied");
    CU(c, cudaSetDevice(c->cfg.device));
    CU(c, cudaStreamSynchronize(c->stream));
    if (c->d2h_stream) CU(c, cudaStreamSynchronize(c->d2h_stream));
    FILE* f = fopen(path, to_file ? "wb" : "rb");
    if (!f) return fail(c, HALOS_ERR_INVALID_ARG, "cannot open %s", path);
    void* bounce = nullptr;
    if (cudaHostAlloc(&bounce, kBounce, cudaHostAllocDefault) != cudaSuccess) {
        (void)cudaGetLastError();
        fclose(f);
        return fail(c, HALOS_ERR_OOM, "pinned bounce buffer allocation failed");
    }
    int rc = HALOS_OK;
    CkptHeader h;
    std::memset(&h, 0, sizeof h);
    std::vector<CkptLps> ls(c->lps.size());
    std::vector<CkptWorker> ws(c->workers.size());
    if (to_file) {
        std::memcpy(h.magic, "HALOSCK1", 8);
        h.version = 2; h.wb = c->wb; h.P = c->P;
        h.n_lps = c->cfg.n_lps; h.n_workers = c->cfg.n_workers; h.n_tensors = c->cfg.n_tensors; h.K = c->cfg.K;
        h.eta_l = c->cfg.eta_l; h.beta_l = c->cfg.beta_l; h.eta_g = c->cfg.eta_g; h.beta_g = c->cfg.beta_g; h.alpha = c->cfg.alpha;
        h.gps_iter = c->gps_iter;
        h.optimizer = c->cfg.optimizer;
        h.delay_l = c->cfg.delay_l;
        h.delay_g = c->cfg.delay_g;
        for (size_t l = 0; l < ls.size(); ++l)
            ls[l] = CkptLps{c->lps[l].t, c->lps[l].t_last, c->lps[l].t_push, c->lps[l].inbox_iter, c->lps[l].phase, 0};
        for (size_t w = 0; w < ws.size(); ++w) ws[w] = CkptWorker{c->workers[w].round, c->workers[w].sched_t};
        if (fwrite(&h, sizeof h, 1, f) != 1 || fwrite(c->tensor_numel.data(), 8, c->tensor_numel.size(), f) != c->tensor_numel.size() ||
            fwrite(ls.data(), sizeof(CkptLps), ls.size(), f) != ls.size() || fwrite(ws.data(), sizeof(CkptWorker), ws.size(), f) != ws.size())
            rc = fail(c, HALOS_ERR_INVALID_ARG, "short write to checkpoint file");
    } else {
        std::vector<uint64_t> numel(c->tensor_numel.size());
        if (fread(&h, sizeof h, 1, f) != 1 || std::memcmp(h.magic, "HALOSCK1", 8) != 0 || h.version != 2)
            rc = fail(c, HALOS_ERR_INVALID_ARG, "not a checkpoint file of this library (or of another version)");
        else if (h.P != c->P || h.wb != c->wb || h.n_lps != c->cfg.n_lps || h.n_workers != c->cfg.n_workers || h.n_tensors != c->cfg.n_tensors ||
                 h.optimizer != c->cfg.optimizer)
            rc = fail(c, HALOS_ERR_INVALID_ARG, "checkpoint shape does not match this context");
        // A run resumed under other hyperparameters is another run: the window length and the delays fix
        // WHEN pushes and momentum refreshes happen, the rates and momenta fix every later value.
        else if (h.K != c->cfg.K || std::memcmp(&h.eta_l, &c->cfg.eta_l, 4) || std::memcmp(&h.beta_l, &c->cfg.beta_l, 4) ||
                 std::memcmp(&h.eta_g, &c->cfg.eta_g, 4) || std::memcmp(&h.beta_g, &c->cfg.beta_g, 4) ||
                 std::memcmp(&h.alpha, &c->cfg.alpha, 4) ||
                 (c->cfg.optimizer == HALOS_OPT_DELAYED_NESTEROV && (h.delay_l != c->cfg.delay_l || h.delay_g != c->cfg.delay_g)))
            rc = fail(c, HALOS_ERR_INVALID_ARG, "checkpoint hyperparameters (K, rates, momenta, alpha, delays) differ from this context's");
        else if (fread(numel.data(), 8, numel.size(), f) != numel.size() || numel != c->tensor_numel)
            rc = fail(c, HALOS_ERR_INVALID_ARG, "checkpoint tensor sizes do not match this context");
        else if (fread(ls.data(), sizeof(CkptLps), ls.size(), f) != ls.size() || fread(ws.data(), sizeof(CkptWorker), ws.size(), f) != ws.size())
            rc = fail(c, HALOS_ERR_INVALID_ARG, "checkpoint file is truncated");
    }
    auto pass = [&](void* dev, size_t bytes) {
        if (rc == HALOS_OK) rc = stream_buffer(c, f, dev, bytes, to_file, bounce);
    };
    pass(c->Theta, c->P * 4);
    pass(c->Mg, c->P * 4);
    if (c->acc_g) pass(c->acc_g, c->P * 4);
    for (auto& s : c->lps) {
        pass(s.th, c->P * 4); pass(s.ml, c->P * 4); pass(s.anchor, c->P * 4); pass(s.outbox, c->P * 4); pass(s.inbox, c->P * 4);
        if (s.acc) pass(s.acc, c->P * 4);
    }
    for (auto& w : c->workers) pass(w.th0, c->P * c->wb);
    if (rc == HALOS_OK && !to_file) {
        c->gps_iter = h.gps_iter;
        for (size_t l = 0; l < ls.size(); ++l) {
            c->lps[l].t = ls[l].t; c->lps[l].t_last = ls[l].t_last; c->lps[l].t_push = ls[l].t_push;
            c->lps[l].inbox_iter = ls[l].inbox_iter; c->lps[l].phase = ls[l].phase;
        }
        for (size_t w = 0; w < ws.size(); ++w) { c->workers[w].round = ws[w].round; c->workers[w].sched_t = ws[w].sched_t; }
    }
    cudaFreeHost(bounce);
    if (fclose(f) != 0 && rc == HALOS_OK && to_file) rc = fail(c, HALOS_ERR_INVALID_ARG, "closing the checkpoint file failed");
    return rc;
}
}  // namespace

int halos_export_file(halos_ctx* c, const char* path) { return checkpoint(c, path, true); }
int halos_import_file(halos_ctx* c, const char* path) { return checkpoint(c, path, false); }

// ------------------------------------------------------------------------------ inspection
static int buffer_of(halos_ctx* c, uint32_t which, uint32_t index, const void** p, uint32_t* elem_bytes) {
    *elem_bytes = 4;
    switch (which) {
        case HALOS_BUF_THETA_G: *p = c->Theta; return HALOS_OK;
        case HALOS_BUF_M_G: *p = c->Mg; return HALOS_OK;
        case HALOS_BUF_THETA_L: case HALOS_BUF_M_L: case HALOS_BUF_ANCHOR: case HALOS_BUF_OUTBOX: case HALOS_BUF_INBOX: {
            if (index >= c->cfg.n_lps) return fail(c, HALOS_ERR_INVALID_ARG, "lps out of range");
            LpsState& s = c->lps[index];
            *p = which == HALOS_BUF_THETA_L ? s.th : which == HALOS_BUF_M_L ? s.ml : which == HALOS_BUF_ANCHOR ? s.anchor
                 : which == HALOS_BUF_OUTBOX ? s.outbox : s.inbox;
            return HALOS_OK;
        }
        case HALOS_BUF_ACC_L:
            if (index >= c->cfg.n_lps || !c->lps[index].acc) return fail(c, HALOS_ERR_INVALID_ARG, "no accumulator (optimizer or lps)");
            *p = c->lps[index].acc;
            return HALOS_OK;
        case HALOS_BUF_ACC_G:
            if (!c->acc_g) return fail(c, HALOS_ERR_INVALID_ARG, "no accumulator with this optimizer");
            *p = c->acc_g;
            return HALOS_OK;
        case HALOS_BUF_THETA0:
            if (index >= c->cfg.n_workers) return fail(c, HALOS_ERR_INVALID_ARG, "worker out of range");
            *p = c->workers[index].th0;
            *elem_bytes = c->wb;
            return HALOS_OK;
    }
    return fail(c, HALOS_ERR_INVALID_ARG, "unknown buffer id %u", which);
}

int halos_peek(halos_ctx* c, uint32_t which, uint32_t index, const void** ptr_dev, uint64_t* numel) {
    if (!c || !ptr_dev) return HALOS_ERR_INVALID_ARG;
    {
        int rq = flush_for(c, which, index);
        if (rq != HALOS_OK) return rq;
    }
    const void* p;
    uint32_t eb;
    int rc = buffer_of(c, which, index, &p, &eb);
    if (rc != HALOS_OK) return rc;
    *ptr_dev = p;
    if (numel) *numel = c->P;
    return HALOS_OK;
}

int halos_read(halos_ctx* c, uint32_t which, uint32_t index, uint64_t offset, uint64_t count, void* dst) {
    if (!c || (!dst && count)) return HALOS_ERR_INVALID_ARG;
    {
        int rq = flush_for(c, which, index);
        if (rq != HALOS_OK) return rq;
    }
    const void* p;
    uint32_t eb;
    int rc = buffer_of(c, which, index, &p, &eb);
    if (rc != HALOS_OK) return rc;
    if (offset > c->P || count > c->P - offset) return fail(c, HALOS_ERR_INVALID_ARG, "range outside the buffer");
    if (count == 0) return HALOS_OK;
    CU(c, cudaSetDevice(c->cfg.device));
    CU(c, cudaMemcpyAsync(dst, (const char*)p + offset * eb, count * eb, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    return HALOS_OK;
}

int halos_counters(halos_ctx* c, uint32_t lps, uint64_t* out) {
    if (!c || !out) return HALOS_ERR_INVALID_ARG;
    if (lps >= c->cfg.n_lps) return fail(c, HALOS_ERR_INVALID_ARG, "lps out of range");
    const LpsState& s = c->lps[lps];
    out[0] = s.t;
    out[1] = s.t_last;
    out[2] = (uint64_t)s.phase;
    out[3] = s.t_push;
    out[4] = c->gps_iter;
    return HALOS_OK;
}

int halos_worker_info(halos_ctx* c, uint32_t worker, uint64_t* out) {
    if (!c || !out) return HALOS_ERR_INVALID_ARG;
    if (worker >= c->cfg.n_workers) return fail(c, HALOS_ERR_INVALID_ARG, "worker out of range");
    out[0] = c->workers[worker].round;
    out[1] = c->workers[worker].sched_t;
    out[2] = c->workers[worker].pending != PEND_NONE;
    return HALOS_OK;
}

int halos_stats(halos_ctx* c, uint32_t what, uint32_t lps, double* out) {
    if (!c || !out) return HALOS_ERR_INVALID_ARG;
    if (!(c->cfg.flags & HALOS_FLAG_STATS)) return fail(c, HALOS_ERR_BAD_STATE, "context was created without HALOS_FLAG_STATS");
    if (what > 2 || lps >= c->cfg.n_lps) return fail(c, HALOS_ERR_INVALID_ARG, "bad statistic or lps");
    const size_t nt = c->tensor_numel.size();
    CU(c, cudaSetDevice(c->cfg.device));
    CU(c, cudaMemcpyAsync(out, c->d_stats + ((size_t)what * c->cfg.n_lps + lps) * nt, nt * 8, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    return HALOS_OK;
}

int halos_stats_log(halos_ctx* c, double* log_dev, uint64_t capacity_records) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (!stats_on(c)) return fail(c, HALOS_ERR_BAD_STATE, "context was created without HALOS_FLAG_STATS");
    if ((log_dev == nullptr) != (capacity_records == 0)) return fail(c, HALOS_ERR_INVALID_ARG, "log pointer and capacity go together");
    if (reinterpret_cast<uintptr_t>(log_dev) & 7) return fail(c, HALOS_ERR_INVALID_ARG, "log not aligned to 8 bytes");
    int rq = flush_all(c);   // queued arrivals belong to the previous log
    if (rq != HALOS_OK) return rq;
    c->stats_log = log_dev;
    c->stats_log_capacity = capacity_records;
    c->stats_seq = 0;
    return HALOS_OK;
}

int halos_info(halos_ctx* c, uint64_t* P, uint32_t* n_tensors, uint32_t* n_chunks, uint64_t* launches) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (P) *P = c->P;
    if (n_tensors) *n_tensors = (uint32_t)c->tensor_numel.size();
    if (n_chunks) *n_chunks = (uint32_t)c->chunks.size();
    if (launches) *launches = c->launches;
    return HALOS_OK;
}

int halos_check_guards(halos_ctx* c, int32_t* first_bad) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (!(c->cfg.flags & HALOS_FLAG_GUARD)) return fail(c, HALOS_ERR_BAD_STATE, "context was created without HALOS_FLAG_GUARD");
    {
        int rq = flush_all(c);
        if (rq != HALOS_OK) return rq;
    }
    CU(c, cudaSetDevice(c->cfg.device));
    CU(c, cudaStreamSynchronize(c->stream));
    int32_t bad = -1;
    std::vector<unsigned char> host;
    for (size_t k = 0; k < c->guards.size() && bad < 0; ++k) {
        const GuardedBuffer& g = c->guards[k];
        const size_t tail = g.padded - g.bytes + kGuardBytes;
        host.resize(kGuardBytes + tail);
        CU(c, cudaMemcpy(host.data(), g.raw, kGuardBytes, cudaMemcpyDeviceToHost));
        CU(c, cudaMemcpy(host.data() + kGuardBytes, g.raw + kGuardBytes + g.bytes, tail, cudaMemcpyDeviceToHost));
        for (unsigned char b : host)
            if (b != 0xA5) {
                bad = (int32_t)k;
                break;
            }
    }
    if (first_bad) *first_bad = bad;
    return HALOS_OK;
}

int halos_batch_info(halos_ctx* c, uint64_t* multi_launches, uint64_t* batched_arrivals) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    if (multi_launches) *multi_launches = c->multi_launches;
    if (batched_arrivals) *batched_arrivals = c->batched_arrivals;
    return HALOS_OK;
}

int halos_timing_enable(halos_ctx* c, int on) {
    if (!c) return HALOS_ERR_INVALID_ARG;
    {
        int rq = flush_all(c);
        if (rq != HALOS_OK) return rq;
    }
    CU(c, cudaSetDevice(c->cfg.device));
    CU(c, cudaStreamSynchronize(c->stream));
    for (auto& t : c->timed) c->event_pool.emplace_back(t.a, t.b);
    c->timed.clear();
    c->timing = on != 0;
    return HALOS_OK;
}

int halos_timing_read(halos_ctx* c, uint32_t kind, uint64_t* launches, double* total_ms) {
    if (!c || kind >= HALOS_K_COUNT) return HALOS_ERR_INVALID_ARG;
    {
        int rq = flush_all(c);
        if (rq != HALOS_OK) return rq;
    }
    CU(c, cudaSetDevice(c->cfg.device));
    CU(c, cudaStreamSynchronize(c->stream));
    uint64_t n = 0;
    double ms = 0.0;
    for (auto& t : c->timed) {
        if (t.kind != (int)kind) continue;
        float x = 0.f;
        CU(c, cudaEventElapsedTime(&x, t.a, t.b));
        ms += x;
        n += 1;
    }
    if (launches) *launches = n;
    if (total_ms) *total_ms = ms;
    return HALOS_OK;
}

int halos_timing_launches(halos_ctx* c, halos_launch_record* out, uint64_t capacity, uint64_t* n_out) {
    if (!c || (!out && capacity)) return HALOS_ERR_INVALID_ARG;
    {
        int rq = flush_all(c);
        if (rq != HALOS_OK) return rq;
    }
    CU(c, cudaSetDevice(c->cfg.device));
    CU(c, cudaStreamSynchronize(c->stream));
    uint64_t n = 0;
    for (auto& t : c->timed) {
        if (n < capacity) {
            float x = 0.f;
            CU(c, cudaEventElapsedTime(&x, t.a, t.b));
            out[n] = halos_launch_record{(uint32_t)t.kind, t.events, t.bytes_per_param, x};
        }
        n += 1;
    }
    if (n_out) *n_out = n;
    return HALOS_OK;
}

const char* halos_strerror(int status) {
    switch (status) {
        case HALOS_OK: return "ok";
        case HALOS_ERR_INVALID_ARG: return "invalid argument";
        case HALOS_ERR_BAD_STATE: return "call order violates the update rules";
        case HALOS_ERR_OOM: return "out of memory";
        case HALOS_ERR_CUDA: return "CUDA error";
        case HALOS_ERR_UNSUPPORTED: return "unsupported";
        case HALOS_ERR_TIMEOUT: return "timed out";
    }
    return "unknown status";
}

const char* halos_last_error(halos_ctx* c) { return c ? c->err.c_str() : g_create_error.c_str(); }

}  // extern "C"

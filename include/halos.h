/* halos.h -- C ABI of the B200 (sm_100a) server-side update path of HALoS
 * (hierarchical asynchronous local SGD).
 *
 * One context holds, on ONE GPU, the state of one global parameter server (GPS), n_lps local
 * parameter servers (LPS) and n_workers workers over P fp32 master parameters:
 *
 *   GPS     Theta (global model), m_g (global momentum), i (GPS iteration)
 *   LPS l   theta (local model), m_l (local momentum), anchor (theta_{t_last}),
 *           outbox (Delta travelling to the GPS), inbox (Theta_i travelling back), t, t_last
 *   worker  theta0 (theta_{t,0}: the model it was last scheduled with), in worker_dtype
 *
 * Every call maps to lines of Algorithm 1 ("HALoS Update Rules") of the paper; ModelUpdate is
 * the momentum rule of Appendix E (update rules of the LPS and the GPS) applied to a
 * displacement d:   m' = beta m + d ;   x' = x + eta [ (1 - beta) d + beta m' ].
 *
 * Conventions
 *  - All state buffers are flat, packed in tensor order (tensor k starts at the sum of the
 *    sizes before it), fp32 except worker snapshots (worker_dtype).  The context OWNS them.
 *  - Pointers named *_dev are device pointers on the context's device, *_host are host pointers.
 *  - All kernels are enqueued on the stream given at creation; calls are asynchronous and stream
 *    ordered.  (Only the host-to-device copies of halos_worker_delta_host run on a second stream
 *    that the context owns; events tie them to the kernels that read them.)  Host-side counters
 *    (t, t_last, i, phases) change at enqueue time.
 *  - Calls that touch the device make the context's device the calling thread's current CUDA device
 *    and leave it so.
 *  - Status HALOS_ERR_CUDA means the CUDA runtime reported an error: treat the context as lost.
 *  - Every call returns a status; on any other status than HALOS_OK (HALOS_ERR_CUDA excepted) the
 *    context's state is unchanged and out-parameters are not written.  Nothing aborts or traps.
 *  - A context is not thread safe.  There is no CPU fallback: without a CUDA device
 *    halos_create fails with HALOS_ERR_CUDA.
 */
#ifndef HALOS_H
#define HALOS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct halos_ctx halos_ctx;

enum {
    HALOS_OK = 0,
    HALOS_ERR_INVALID_ARG = 1,
    HALOS_ERR_BAD_STATE = 2,   /* call order violates Algorithm 1 (e.g. pull before the GPS answered) */
    HALOS_ERR_OOM = 3,
    HALOS_ERR_CUDA = 4,
    HALOS_ERR_UNSUPPORTED = 5,
    HALOS_ERR_TIMEOUT = 6      /* reserved for calls that wait on a device-side flag; no call of this build does */
};

enum { HALOS_F32 = 0, HALOS_BF16 = 1 };

/* Server-side optimizer.
 * HALOS_OPT_PAPER: the ModelUpdate rule the paper defines (Appendix E); the default.
 * HALOS_OPT_DELAYED_NESTEROV: the optimizer the paper's experiments used ("delayed Nesterov", cited from
 * the Async-Local-SGD work, never defined in the paper; the footnote of its hyperparameter table in
 * Appendix D only states that the rule scales the step by 1/delay).  Reading implemented, per server
 * with delay n, rate eps (= eta_l / eta_g), accumulator acc, k = number of updates seen so far:
 *     acc += d                                            every update (d = displacement)
 *     k mod n != 0:   x += (eps/n) d                      momentum untouched
 *     k mod n == 0:   m = beta m + acc/n ;  x += eps (beta m + d/n) ;  acc = 0
 * The paper's selected values in this mode: delay_l = 16, eta_l = 3.2, delay_g = 2, eta_g = 0.3. */
enum { HALOS_OPT_PAPER = 0, HALOS_OPT_DELAYED_NESTEROV = 1 };

/* flags */
enum {
    HALOS_FLAG_STATS = 1u,         /* keep per-tensor squared norms of delta, theta_t (arrive) and Delta (push); formed in
                                      registers by the update kernels, in every mode (fused launches, both optimizers,
                                      materialised deltas); needs chunk_elems <= 8192 */
    HALOS_FLAG_MATERIALISE_DELTA = 2u, /* halos_worker_delta forms delta (fp32) into a context buffer at once, so the
                                          borrow of theta_H ends when that call has been enqueued; costs one 4P
                                          buffer per worker and 4 + 2 w_b extra bytes of traffic per parameter */
    HALOS_FLAG_GUARD = 4u          /* surround every state buffer with 256-byte canary zones (halos_check_guards) */
};

/* LPS phase of the push / merge round trip */
enum { HALOS_IDLE = 0, HALOS_PUSHED = 1, HALOS_ANSWERED = 2 };

/* buffers addressable through halos_peek / halos_read */
enum {
    HALOS_BUF_THETA_G = 0,  /* Theta          (index ignored) */
    HALOS_BUF_M_G = 1,      /* m_g            (index ignored) */
    HALOS_BUF_THETA_L = 2,  /* theta  of LPS index */
    HALOS_BUF_M_L = 3,      /* m_l    of LPS index */
    HALOS_BUF_ANCHOR = 4,   /* theta_{t_last} of LPS index */
    HALOS_BUF_OUTBOX = 5,   /* Delta in flight from LPS index */
    HALOS_BUF_INBOX = 6,    /* Theta_i in flight to LPS index */
    HALOS_BUF_THETA0 = 7,   /* start snapshot of worker index (worker_dtype) */
    HALOS_BUF_ACC_L = 8,    /* delayed Nesterov accumulator of LPS index  (that optimizer only) */
    HALOS_BUF_ACC_G = 9     /* delayed Nesterov accumulator of the GPS    (that optimizer only) */
};

typedef struct halos_config {
    uint32_t struct_size;          /* = sizeof(halos_config); checked */
    uint32_t n_lps;
    uint32_t n_workers;
    const uint32_t* worker_lps;    /* host, [n_workers]: LPS of each worker; copied */
    uint32_t n_tensors;
    const uint64_t* tensor_numel;  /* host, [n_tensors]: elements per tensor; copied; sum = P */
    float eta_l, beta_l;           /* local learning rate and momentum  (paper's selection: 0.2, 0.9) */
    float eta_g, beta_g;           /* global learning rate and momentum (0.15, 0.5) */
    float alpha;                   /* merging weight (0.25) */
    uint32_t K;                    /* local updates accumulated per push (32) */
    uint32_t worker_dtype;         /* HALOS_F32 | HALOS_BF16: type of theta0 snapshots and theta_H inputs */
    uint32_t flags;
    int32_t device;                /* CUDA device ordinal */
    void* stream;                  /* cudaStream_t; NULL = the legacy default stream */
    /* Optional device allocator (e.g. a shim over the PyTorch caching allocator).  NULL = cudaMalloc /
     * cudaFree.  alloc returns a device pointer aligned to >= 256 bytes or NULL. */
    void* (*alloc)(size_t bytes, void* user);
    void (*free_)(void* ptr, void* user);
    void* alloc_user;
    uint32_t chunk_elems;          /* scheduler chunk size in elements; 0 = library default */
    uint32_t optimizer;            /* HALOS_OPT_PAPER | HALOS_OPT_DELAYED_NESTEROV */
    uint32_t delay_l, delay_g;     /* momentum refresh interval of the LPSs / the GPS (delayed Nesterov; >= 1) */
    uint32_t reserved;
} halos_config;

/* Fills *cfg with the paper's selected hyperparameters and library defaults (everything else zero). */
void halos_default_config(halos_config* cfg);

/* Alg. 1 lines 6-7 (initialisation): Theta = theta[l] = anchor[l] = Theta_0, theta0[w] = cast(Theta_0),
 * momenta 0, t = t_last = i = 0.  theta_init_dev: device, P fp32, flat, borrowed during the call only
 * (the call synchronises the stream before returning).  *out receives the context. */
int halos_create(const halos_config* cfg, const float* theta_init_dev, halos_ctx** out);

/* Alg. 1 line 25 (worker side, delta = theta_{t,H} - theta_{t,0}).  Registers the result theta_{t,H}
 * of `worker`; the subtraction itself is fused into the next halos_lps_apply for this worker so
 * delta never touches memory.  Exactly one of thetaH_flat_dev (device, P elements of worker_dtype,
 * packed like the state) and thetaH_ptrs_host (host array of n_tensors DEVICE pointers, one per
 * tensor, each tensor contiguous) is non-NULL.  The device data is BORROWED until the matching
 * halos_lps_apply has completed in stream order -- or, on a context created with
 * HALOS_FLAG_MATERIALISE_DELTA, only until the work this call enqueues has completed (delta is then
 * written to a context buffer by a kernel of its own and halos_lps_apply reads that buffer; the
 * resulting state is bit-identical).  BAD_STATE if the worker already has a pending result. */
int halos_worker_delta(halos_ctx* ctx, uint32_t worker, const void* thetaH_flat_dev,
                       const void* const* thetaH_ptrs_host);

/* Same, for a result that sits in HOST memory (P elements of worker_dtype, packed): it is copied
 * into one of two context-owned staging buffers (allocated on first use) by a copy stream the
 * context owns, ordered against the update kernels with events, so that the copy of the next result
 * overlaps the kernel of the current one; pinned host memory makes the copy asynchronous.  The host
 * data is borrowed until that copy has completed.  BAD_STATE if both staging buffers still hold
 * results that were not applied (at most two host results may be pending), OOM if a staging buffer
 * cannot be allocated. */
int halos_worker_delta_host(halos_ctx* ctx, uint32_t worker, const void* thetaH_flat_host);

/* Alg. 1 line 12 seen from the worker: the model the worker restarts from, theta_{t,0} = cast(theta_t), as
 * written by its last halos_lps_apply, copied to HOST memory (P elements of worker_dtype, packed).  The copy
 * runs on a device-to-host stream the context owns, after the update that wrote the snapshot and before
 * the next one that rewrites it (events order both), so it overlaps the update kernels and the host-to-device
 * copies of halos_worker_delta_host.  dst_host is borrowed until halos_fetch_sync returns (pinned memory
 * makes the copy asynchronous).  Launches a queued arrival of this worker first. */
int halos_worker_fetch_host(halos_ctx* ctx, uint32_t worker, void* dst_host);
/* Waits until every copy enqueued by halos_worker_fetch_host has landed in host memory. */
int halos_fetch_sync(halos_ctx* ctx);

/* Alg. 1 lines 10-13 at LPS `lps` for the pending result of `worker`:  t <- t+1;
 * theta_t <- ModelUpdate(theta_{t-1}, delta, eta_l, beta_l); the worker is scheduled theta_t
 * (theta0[worker] <- cast(theta_t)).  One fused kernel.  *push_due (may be NULL) receives
 * (t - t_last == K).  INVALID_ARG if the worker does not belong to lps; BAD_STATE if it has no
 * pending result. */
int halos_lps_apply(halos_ctx* ctx, uint32_t lps, uint32_t worker, int* push_due);

/* Alg. 1 line 14: outbox[lps] <- Delta = theta_t - theta_{t_last}.  The LPS goes on updating while
 * Delta is in flight.  BAD_STATE if a round trip is already in flight for this LPS.  The library
 * does not insist on t - t_last == K; the caller (halos_replay) decides when to push. */
int halos_lps_push(halos_ctx* ctx, uint32_t lps);

/* Alg. 1 lines 2-4: the GPS receives outbox[lps]; i <- i+1; Theta_i <- ModelUpdate(Theta_{i-1}, Delta,
 * eta_g, beta_g); inbox[lps] <- Theta_i (a snapshot).  BAD_STATE unless lps has pushed. */
int halos_gps_merge(halos_ctx* ctx, uint32_t lps);

/* Alg. 1 lines 18-19: t_last <- t; theta_t <- (1-alpha) theta_t + alpha inbox[lps]; anchor <- theta_t.
 * BAD_STATE unless the GPS has answered this LPS. */
int halos_lps_pull(halos_ctx* ctx, uint32_t lps);

/* Alg. 1 lines 2-4 directly followed by lines 17-20 for the same LPS, as one launch: exactly
 * halos_gps_merge(lps) then halos_lps_pull(lps) -- same state afterwards, bit for bit, inbox included --
 * with Theta_i merged from registers (36 instead of 40 bytes of traffic per parameter).  For a queue in
 * which the answer of the GPS is the very next message this LPS processes (Sec. 4.1: one queue per
 * server, processed in order).  BAD_STATE unless lps has pushed. */
int halos_gps_merge_pull(halos_ctx* ctx, uint32_t lps);

/* Synchronises the stream and frees everything the context owns.  NULL is accepted. */
int halos_destroy(halos_ctx* ctx);

/* ------------------------------------------------------------------ auxiliary calls ----------- */

/* Event-queue driver (the single queue of Sec. 4.1: worker results and global models are processed
 * in arrival order; Appendix A: the trace is replayed in its recorded order). */
enum { HALOS_EV_ARRIVE = 0, HALOS_EV_GPS_RECV = 1, HALOS_EV_PULL = 2 };

typedef struct halos_event {
    uint8_t kind;      /* HALOS_EV_* */
    uint8_t lps;
    uint16_t worker;   /* ARRIVE only */
    uint32_t pad;
    int64_t time_ns;   /* informational */
} halos_event;

typedef struct halos_event_log {
    uint32_t index;            /* position in the trace */
    uint8_t kind, lps;
    uint16_t worker;
    uint64_t t, t_last;        /* LPS counters after the event */
    uint64_t gps_iter;         /* GPS iteration i after the event */
    uint64_t worker_staleness; /* ARRIVE: LPS updates applied since this worker was scheduled */
    uint64_t gps_lag;          /* PULL: GPS iterations since the merged Theta_i was produced */
    uint8_t pushed;            /* ARRIVE: this arrival completed a window of K and pushed */
    uint8_t fused;             /* the event ran inside a fused launch */
    uint8_t pad[6];
} halos_event_log;

/* Called by halos_replay before each ARRIVE to obtain the worker's result theta_{t,H}: fill exactly
 * one of *flat_dev / *ptrs_host (same meaning as in halos_worker_delta).  `round` counts this
 * worker's arrivals from 0.  Any work the producer enqueues must go to the context's stream.
 * Return 0, or nonzero to abort the replay. */
typedef int (*halos_producer_fn)(void* user, uint32_t event_index, uint32_t worker, uint64_t round,
                                 const void** flat_dev, const void* const** ptrs_host);

/* Replays events[0..n) in order: ARRIVE = worker_delta + lps_apply (+ lps_push when the window of
 * K closes, fused into the same launch), GPS_RECV = gps_merge, PULL = lps_pull (with max_batch > 1, a
 * GPS_RECV directly followed by the PULL of the same LPS runs as halos_gps_merge_pull).  log_host (may be
 * NULL) receives one record per event.  Stops at the first failing event: returns its status and
 * writes its index to *failed_at (may be NULL); events before it stay applied.  An ARRIVE that cannot be
 * applied (worker of another LPS; window due while a round trip is in flight) is refused BEFORE the
 * producer is asked, so a failed replay never leaves a borrowed result registered. */
int halos_replay(halos_ctx* ctx, const halos_event* events_host, uint32_t n, halos_producer_fn producer,
                 void* user, halos_event_log* log_host, uint32_t* failed_at);

/* The same replay with multi-event fusion: up to max_batch (<= 8) arrivals at one LPS, from distinct
 * workers, are applied by ONE kernel that reads and writes that LPS's model and momentum once for
 * the whole batch (per element the updates are applied in queue order, so the state after the call
 * is bit-identical to halos_replay, and so is the log except for its `fused` flags).  Counters, the
 * log and the producer calls still follow trace order; only kernel launches are deferred, past events
 * that touch disjoint buffers.  Consequence for the producer: a result it returned must stay valid
 * until the producer is called again for the SAME worker or the replay returns (with halos_replay it
 * only has to survive until the next producer call).  max_batch <= 1 behaves like halos_replay.
 * Statistics (HALOS_FLAG_STATS) are kept per arrival inside fused launches and equal those of the
 * unfused replay bit for bit (arrivals whose tensors differ in vector alignment are not fused). */
int halos_replay_batched(halos_ctx* ctx, const halos_event* events_host, uint32_t n, halos_producer_fn producer,
                         void* user, halos_event_log* log_host, uint32_t* failed_at, uint32_t max_batch);

/* Streaming form of halos_replay_batched for a queue that is fed call after call: arrivals still
 * waiting for companions when the call returns STAY queued (their counters are already advanced, their
 * kernels not yet launched) and may be fused with arrivals of the next call.  They are launched by the
 * next call that needs them, by halos_flush, and by every other entry point that reads or changes
 * the state they touch (lps_apply, lps_push, lps_pull, export/import, timing, destroy; peek and read
 * launch the queue of the LPS or worker whose buffer is asked for).  A result
 * returned by the producer must stay valid until the same worker's next producer call or the next
 * halos_flush, whichever comes first. */
int halos_replay_stream(halos_ctx* ctx, const halos_event* events_host, uint32_t n, halos_producer_fn producer,
                        void* user, halos_event_log* log_host, uint32_t* failed_at, uint32_t max_batch);

/* The same drivers for results that already exist (a stored trace replayed with its stored results, or a
 * backlog of results that arrived while the server was busy): results_host[k] is the flat device pointer
 * (P elements of worker_dtype) of event k if it is an ARRIVE and ignored otherwise; no callback is made.
 * keep_queued = 0 behaves like halos_replay_batched, nonzero like halos_replay_stream; the borrow rules are
 * those of the respective call (a result must stay valid until the same worker's next arrival has been
 * launched, the replay has returned, or -- streaming -- halos_flush).  A NULL entry for an ARRIVE fails
 * that event with INVALID_ARG.  The host cost per event is one kernel launch at most, which matters for
 * models small enough to be launch-bound. */
int halos_replay_results(halos_ctx* ctx, const halos_event* events_host, uint32_t n, const void* const* results_host,
                         halos_event_log* log_host, uint32_t* failed_at, uint32_t max_batch, int keep_queued);

/* Launches every arrival that halos_replay_stream left queued. */
int halos_flush(halos_ctx* ctx);

/* Read-only device pointer to a state buffer (for inspection; valid until halos_destroy).
 * *numel = P.  Element type fp32, or worker_dtype for HALOS_BUF_THETA0. */
int halos_peek(halos_ctx* ctx, uint32_t which, uint32_t index, const void** ptr_dev, uint64_t* numel);

/* Copies elements [offset, offset+count) of a state buffer to host memory, in stream order, and
 * waits for the copy. */
int halos_read(halos_ctx* ctx, uint32_t which, uint32_t index, uint64_t offset, uint64_t count,
               void* dst_host);

/* counters_host[5] = { t, t_last, phase, t at the last push, GPS iteration i } for one LPS. */
int halos_counters(halos_ctx* ctx, uint32_t lps, uint64_t* counters_host);

/* info_host[3] = { arrivals seen from the worker, LPS counter t when it was last scheduled, pending } */
int halos_worker_info(halos_ctx* ctx, uint32_t worker, uint64_t* info_host);

/* Per-tensor squared norms (needs HALOS_FLAG_STATS): what = 0: sum delta^2 of the last
 * halos_lps_apply of this LPS; what = 1: sum Delta^2 of its last halos_lps_push; what = 2: sum theta_t^2 of
 * its model right after that last halos_lps_apply.  After a fused launch "last" is the last arrival of the
 * batch.  The sums are reduced in a fixed order that depends on neither the launch configuration nor the
 * number of fused arrivals.  Waits for the stream.  out_host: [n_tensors] doubles. */
int halos_stats(halos_ctx* ctx, uint32_t what, uint32_t lps, double* out_host);

/* Per-arrival statistics log (needs HALOS_FLAG_STATS).  log_dev: caller-owned device array of
 * capacity_records records of 3 * n_tensors doubles; from now on the r-th arrival accounted for on this
 * context (r from 0, in trace order, however its launch is fused or deferred) fills record r with
 * [sum delta^2 per tensor | sum theta_t^2 per tensor | sum Delta^2 per tensor (zeros unless the arrival
 * closed a window and its push was fused)] in stream order; arrivals beyond the capacity are not recorded.
 * NULL / 0 detaches.  The array is borrowed until detached or the context is destroyed. */
int halos_stats_log(halos_ctx* ctx, double* log_dev, uint64_t capacity_records);

/* Number of parameters P, tensors, scheduler chunks, and kernels launched so far. */
int halos_info(halos_ctx* ctx, uint64_t* P, uint32_t* n_tensors, uint32_t* n_chunks, uint64_t* launches);

/* Checkpoint / resume.  halos_export_file writes the whole state (every buffer, all counters and
 * phases) to a file; halos_import_file loads it into a context that was created with the same
 * shape (P, tensors, servers, workers, worker_dtype, optimizer) and the same hyperparameters (K, eta_l,
 * beta_l, eta_g, beta_g, alpha bit for bit, and delay_l / delay_g under delayed Nesterov) -- all checked,
 * a mismatch is INVALID_ARG and leaves the context untouched -- and replaces its state, so that a
 * replay continued after export -> destroy -> create -> import equals the uninterrupted replay bit
 * for bit.  Both wait for the stream.  BAD_STATE if any worker result is registered but not yet
 * applied (borrowed caller memory cannot be checkpointed); INVALID_ARG on I/O errors or a file
 * that does not match. */
int halos_export_file(halos_ctx* ctx, const char* path);
int halos_import_file(halos_ctx* ctx, const char* path);

/* Out-of-bounds write detector for test runs (needs HALOS_FLAG_GUARD): waits for the stream and checks
 * the canary bytes around every state buffer.  *first_bad = -1 if all are intact, else the index of the
 * first damaged buffer in allocation order (Theta, m_g, [acc_g], then per LPS theta, m_l, anchor, outbox,
 * inbox, [acc], then per worker its snapshot [and its materialised delta]). */
int halos_check_guards(halos_ctx* ctx, int32_t* first_bad);

/* Multi-event fusion counters since creation: launches of the multi-arrival kernel and the number
 * of arrivals they covered (algorithmic bytes of those launches: (16 launches + 3 w_b arrivals) P). */
int halos_batch_info(halos_ctx* ctx, uint64_t* multi_launches, uint64_t* batched_arrivals);

/* Per-kernel device timing.  While enabled, every update kernel is bracketed by CUDA events on the
 * context's stream; halos_timing_read waits for the stream and returns, for one kernel kind, how
 * many launches were timed since halos_timing_enable(ctx, 1) and their summed duration. */
enum {
    HALOS_K_ARRIVE = 0,       /* delta + LPS momentum update + schedule copy */
    HALOS_K_ARRIVE_PUSH = 1,  /* the same, plus Delta formed in the same pass */
    HALOS_K_PUSH = 2,
    HALOS_K_GPS = 3,          /* global momentum update + Theta_i snapshot */
    HALOS_K_PULL = 4,         /* merge + anchor reset */
    HALOS_K_ARRIVE_MULTI = 5, /* 2-8 arrivals at one LPS in one pass (halos_replay_batched) */
    HALOS_K_GPS_PULL = 6,     /* GPS update + merge into the same LPS in one pass (halos_gps_merge_pull) */
    HALOS_K_COUNT = 7
};
int halos_timing_enable(halos_ctx* ctx, int on);
int halos_timing_read(halos_ctx* ctx, uint32_t kind, uint64_t* launches, double* total_ms);

/* One record per launch timed since halos_timing_enable(ctx, 1), in launch order: its kind, how many trace
 * events it carried out (a fused launch: several), its algorithmic traffic in bytes per parameter (every
 * live buffer read once and written once: 16 + 3 w_b per arrival alone, 16 + 3 w_b n for n fused arrivals,
 * +8 with Delta formed in the same pass, +8 for a momentum refresh under delayed Nesterov, 12 push, 24 GPS,
 * 16 merge, 36 GPS+merge) and its duration.  Waits for the stream.  *n receives the number of launches
 * timed; at most `capacity` records are written. */
typedef struct halos_launch_record {
    uint32_t kind;             /* HALOS_K_* */
    uint32_t events;
    uint32_t bytes_per_param;
    float ms;
} halos_launch_record;
int halos_timing_launches(halos_ctx* ctx, halos_launch_record* out_host, uint64_t capacity, uint64_t* n);

/* Push step for callers that must not allocate.  (The paper has no counterpart: this is a
 * deployment variant of Alg. 1 line 14 as computed by halos_lps_push with HALOS_FLAG_STATS.)
 *
 *   Delta_dev[j] = theta_dev[j] - anchor_dev[j]  for j < n,   *sqnorm_dev = sum_j Delta_dev[j]^2
 *
 * Meant for code that runs where device allocation is off limits: while a memory pool is frozen
 * or full, in sections where an allocator call could block or synchronise the device, or under a
 * policy of no cudaMalloc after start-up.  It needs no context; inputs and outputs are the caller's
 * (device pointers on `device`, fp32 arrays of n elements, 4-byte aligned -- 16-byte alignment of all
 * three enables the vector path; sqnorm_dev points to one double).  The reduction scratch is a fixed
 * 512 KB array inside the library, present on every GPU that loads it until the process exits, which
 * caps n at HALOS_NOALLOC_MAX_ELEMS: larger n returns HALOS_ERR_UNSUPPORTED and touches nothing.
 * Once warmed up, a call allocates nothing (no cudaMalloc/cudaFree, no allocating library routine) and
 * enqueues two kernels on `stream` (cudaStream_t, NULL = legacy default stream); it does not wait for them.
 * Warm-up: the FIRST call on each device may create that device's primary context, loads the two kernels
 * and the scratch array with them (the runtime takes device memory for this) and looks up the array's
 * device address (cudaGetSymbolAddress).  Make that call -- n = 0 is enough -- at start-up, while
 * allocation is still allowed and before any stream capture begins; later calls on that device touch no
 * allocator.  Every call makes `device` the calling thread's current CUDA device and leaves it so.
 * All calls share the scratch,
 * which keeps the previous call's partial sums; each call overwrites every slot it later reads, so
 * nothing needs clearing, but calls that overlap on the GPU race on it: keep them on one stream or
 * otherwise serialised.  Returns HALOS_OK, HALOS_ERR_UNSUPPORTED (n too large),
 * HALOS_ERR_INVALID_ARG (null pointer, array not 4-byte aligned, sqnorm_dev not 8-byte aligned, bad
 * device; checked on the host before anything is launched) or HALOS_ERR_CUDA. */
#define HALOS_NOALLOC_MAX_ELEMS (1ull << 29)
int halos_push_noalloc(int32_t device, void* stream, const float* theta_dev, const float* anchor_dev,
                       float* Delta_dev, uint64_t n, double* sqnorm_dev);

const char* halos_strerror(int status);
/* Text of the last error on this context (or of the last failed halos_create when ctx is NULL). */
const char* halos_last_error(halos_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* HALOS_H */

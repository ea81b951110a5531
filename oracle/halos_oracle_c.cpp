// C entry points around the CPU oracle so that Python tests can drive it through ctypes.
// Test infrastructure only: nothing in the CUDA library links or loads this file.
#include "halos_oracle.hpp"

#include <chrono>
#include <cstdio>
#include <thread>

using namespace halos_oracle;

namespace {
struct Handle {
    int is_double;
    Oracle<float>* f;
    Oracle<double>* d;
    char err[256];
};

template <class F>
int guarded(Handle* h, F&& fn) {
    try {
        fn();
        return 0;
    } catch (const std::exception& e) {
        if (h) std::snprintf(h->err, sizeof h->err, "%s", e.what());
        return 1;
    }
}
}  // namespace

extern "C" {

// which: 0 Theta, 1 Mg, 2 th[l], 3 ml[l], 4 anchor[l], 5 outbox[l], 6 inbox[l], 7 th0[w], 8 last delta[l], 9 acc[l], 10 acc_g
enum { B_THETA = 0, B_MG, B_TH, B_ML, B_ANCHOR, B_OUTBOX, B_INBOX, B_TH0, B_DELTA, B_ACC_L, B_ACC_G };

void* halos_oracle_create(int use_double, uint64_t P, uint32_t n_lps, uint32_t n_workers,
                          const uint32_t* worker_lps, double eta_l, double beta_l, double eta_g,
                          double beta_g, double alpha, uint32_t K, int worker_dtype,
                          const float* theta_init, int optimizer, uint32_t delay_l, uint32_t delay_g) {
    Config c;
    c.P = P;
    c.n_lps = n_lps;
    c.n_workers = n_workers;
    c.worker_lps.assign(worker_lps, worker_lps + n_workers);
    c.eta_l = eta_l;
    c.beta_l = beta_l;
    c.eta_g = eta_g;
    c.beta_g = beta_g;
    c.alpha = alpha;
    c.K = K;
    c.worker_dtype = worker_dtype;
    c.optimizer = optimizer;
    c.delay_l = delay_l;
    c.delay_g = delay_g;
    Handle* h = new Handle();
    h->is_double = use_double;
    h->f = nullptr;
    h->d = nullptr;
    h->err[0] = 0;
    try {
        if (use_double)
            h->d = new Oracle<double>(c, theta_init);
        else
            h->f = new Oracle<float>(c, theta_init);
    } catch (const std::exception& e) {
        std::fprintf(stderr, "halos_oracle_create: %s\n", e.what());
        delete h;
        return nullptr;
    }
    return h;
}

void halos_oracle_destroy(void* hv) {
    Handle* h = (Handle*)hv;
    if (!h) return;
    delete h->f;
    delete h->d;
    delete h;
}

const char* halos_oracle_error(void* hv) { return ((Handle*)hv)->err; }

// returns 0 ok / 1 error; *pushed = 1 if the arrival closed a window of K updates
int halos_oracle_arrive(void* hv, uint32_t w, const void* thetaH, int* pushed) {
    Handle* h = (Handle*)hv;
    return guarded(h, [&] {
        bool p = h->is_double ? h->d->arrive(w, thetaH) : h->f->arrive(w, thetaH);
        if (pushed) *pushed = p ? 1 : 0;
    });
}
// Alg. 1 line 14 on its own (tests that push at times other than the window of K)
int halos_oracle_push(void* hv, uint32_t l) {
    Handle* h = (Handle*)hv;
    return guarded(h, [&] { h->is_double ? h->d->push(l) : h->f->push(l); });
}
int halos_oracle_gps_recv(void* hv, uint32_t l) {
    Handle* h = (Handle*)hv;
    return guarded(h, [&] { h->is_double ? h->d->gps_recv(l) : h->f->gps_recv(l); });
}
int halos_oracle_pull(void* hv, uint32_t l) {
    Handle* h = (Handle*)hv;
    return guarded(h, [&] { h->is_double ? h->d->pull(l) : h->f->pull(l); });
}

// Pointer to the oracle's own storage of one buffer (element type: T for master buffers;
// float or uint16 for worker snapshots).  Valid until destroy.
void* halos_oracle_buffer(void* hv, int which, uint32_t idx) {
    Handle* h = (Handle*)hv;
    auto pick = [&](auto* o) -> void* {
        switch (which) {
            case B_THETA: return o->Theta.data();
            case B_MG: return o->Mg.data();
            case B_TH: return idx < o->lps.size() ? o->lps[idx].th.data() : nullptr;
            case B_ML: return idx < o->lps.size() ? o->lps[idx].ml.data() : nullptr;
            case B_ANCHOR: return idx < o->lps.size() ? o->lps[idx].anchor.data() : nullptr;
            case B_OUTBOX: return idx < o->lps.size() ? o->lps[idx].outbox.data() : nullptr;
            case B_INBOX: return idx < o->lps.size() ? o->lps[idx].inbox.data() : nullptr;
            case B_ACC_L: return idx < o->lps.size() ? o->lps[idx].acc.data() : nullptr;
            case B_ACC_G: return o->acc_g.data();
            case B_DELTA: return idx < o->lps.size() ? o->lps[idx].last_delta.data() : nullptr;
            case B_TH0:
                if (idx >= o->cfg.n_workers) return nullptr;
                return o->cfg.worker_dtype == W_F32 ? (void*)o->th0_f32[idx].data()
                                                    : (void*)o->th0_bf16[idx].data();
        }
        return nullptr;
    };
    return h->is_double ? pick(h->d) : pick(h->f);
}

// counters: out[0]=t, out[1]=t_last, out[2]=phase, out[3]=t_push for LPS l; out[4]=GPS i
void halos_oracle_counters(void* hv, uint32_t l, uint64_t* out) {
    Handle* h = (Handle*)hv;
    auto fill = [&](auto* o) {
        out[0] = o->lps.at(l).t;
        out[1] = o->lps.at(l).t_last;
        out[2] = (uint64_t)o->lps.at(l).phase;
        out[3] = o->lps.at(l).t_push;
        out[4] = o->i;
    };
    if (h->is_double)
        fill(h->d);
    else
        fill(h->f);
}

// worker bookkeeping: out[0] = arrivals seen from w, out[1] = LPS counter t when w was last scheduled
void halos_oracle_worker(void* hv, uint32_t w, uint64_t* out) {
    Handle* h = (Handle*)hv;
    auto fill = [&](auto* o) {
        out[0] = o->worker_round.at(w);
        out[1] = o->worker_sched_t.at(w);
    };
    if (h->is_double)
        fill(h->d);
    else
        fill(h->f);
}

// bf16 conversion helpers exposed for the rounding tests
uint16_t halos_oracle_f32_to_bf16(float x) { return f32_to_bf16_rne(x); }
float halos_oracle_bf16_to_f32(uint16_t h) { return bf16_to_f32(h); }

}  // extern "C"

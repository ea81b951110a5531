// HALoS server-side update rules -- CPU ORACLE (test infrastructure, not product code).
//
// A plain, sequential, one-element-at-a-time implementation of the update rules of
// Algorithm 1 ("HALoS Update Rules") with ModelUpdate as defined in Appendix E
// ("Proof of Theorem 4.6", the LPS and GPS momentum rules).  It exists only so that the
// CUDA library can be checked against it: tests, the smoke check and the benchmark's CPU
// baseline leg are its only callers.  It shares no code with the CUDA path.
//
// Scalar type T: float is the parity oracle (the CUDA path computes in fp32 and every
// rounding below is mirrored there), double is the self-check oracle that is pinned to
// closed forms and exact hand expansions.
//
// State, in the paper's notation:
//   GPS:  Theta (global model Theta_i), Mg (global momentum m_g), i (GPS iteration)
//   LPS l: th (theta_t), ml (local momentum m_l), anchor (theta_{t_last}),
//          outbox (Delta in flight to the GPS), inbox (Theta_i in flight back), t, t_last
//   worker w: th0 (theta_{t,0}, the model the worker was last scheduled with), stored in
//          the worker dtype (fp32, or bf16 as 16-bit patterns)
//
// Readings taken where the paper leaves a choice (all stated again in the design notes):
//   * ModelUpdate receives displacements (delta = theta_{t,H} - theta_{t,0}, Alg. 1 line 25;
//     Delta = theta_t - theta_{t_last}, line 14) while Appendix E writes it for a gradient
//     with a minus sign.  A displacement is minus a pseudo-gradient, so the step is ADDED:
//       m' = beta m + d ;  theta' = theta + eta [ (1-beta) d + beta m' ].
//   * Momenta start at zero.
//   * theta_{t_last} is the LPS model AFTER the merge of line 19 (line 18 sets t_last <- t
//     and line 19 then redefines theta_t), so Delta holds exactly the K worker updates
//     applied since the merge.
//   * The GPS applies one LPS's Delta per iteration (Alg. 1 lines 2-3), no 1/M average.
//   * Delta is not divided by K.
//   * Rounding order: each fma below is one fused multiply-add (single rounding); every
//     other product or difference is rounded on its own.  Compile with -ffp-contract=off.
//
// Optional optimizer OPT_DELAYED_NESTEROV.  The paper's experiments replace ModelUpdate by the
// "delayed Nesterov" optimizer of the Async-Local-SGD work it cites, but never define it; the only
// property it states (footnote of the hyperparameter table, Appendix D) is that the rule scales the
// step by 1/delay.  The reading implemented here, per server with delay d,
// rate eps, an accumulator acc and n = number of updates seen so far:
//     acc += g                                        every update
//     n mod d != 0:  theta -= (eps/d) g               momentum untouched
//     n mod d == 0:  m = beta m + acc/d ;  theta -= eps (beta m + g/d) ;  acc = 0
// (g = -displacement as above).  THE READING IS UNPINNED BY THE PAPER; the implementation is
// pinned to the stated property (mean step eps g / (d (1-beta)) under constant g), to textbook
// Nesterov SGD for d = 1, and to an independent interpreter.
#pragma once
#include <cmath>
#include <cstdint>
#include <cstring>
#include <stdexcept>
#include <vector>

namespace halos_oracle {

enum WorkerDtype { W_F32 = 0, W_BF16 = 1 };
enum Phase { IDLE = 0, PUSHED = 1, ANSWERED = 2 };
enum Optimizer { OPT_PAPER = 0, OPT_DELAYED_NESTEROV = 1 };

// fp32 -> bf16, round to nearest, ties to even; result is the upper 16 bits.
// Written out on integers so that it does not depend on any hardware conversion.
inline uint16_t f32_to_bf16_rne(float x) {
    uint32_t u;
    std::memcpy(&u, &x, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);  // NaN stays NaN
    uint32_t lower = u & 0xffffu;
    uint32_t upper = u >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1u;  // may carry into the exponent: correct
    return (uint16_t)upper;
}
inline float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float x;
    std::memcpy(&x, &u, 4);
    return x;
}

struct Config {
    uint64_t P = 0;                    // parameters
    uint32_t n_lps = 0, n_workers = 0;
    std::vector<uint32_t> worker_lps;  // worker -> its LPS
    double eta_l = 0.2, beta_l = 0.9;  // local learning rate / momentum  (hyperparameter table, Appendix D)
    double eta_g = 0.15, beta_g = 0.5; // global learning rate / momentum
    double alpha = 0.25;               // merging weight
    uint32_t K = 32;                   // local updates accumulated per push
    int worker_dtype = W_F32;
    int optimizer = OPT_PAPER;
    uint32_t delay_l = 1, delay_g = 1;  // momentum refresh interval of the LPSs / the GPS (delayed Nesterov only)
};

template <class T>
struct Lps {
    std::vector<T> th, ml, anchor, outbox, inbox;
    std::vector<T> last_delta;  // the worker displacement applied by the most recent arrival (observability)
    std::vector<T> acc;         // delayed Nesterov: displacements accumulated since the last momentum refresh
    uint64_t t = 0, t_last = 0, t_push = 0;
    int phase = IDLE;
};

template <class T>
class Oracle {
public:
    Config cfg;
    std::vector<T> Theta, Mg;
    std::vector<T> acc_g;  // delayed Nesterov accumulator of the GPS
    uint64_t i = 0;
    std::vector<Lps<T>> lps;
    std::vector<std::vector<float>> th0_f32;      // worker snapshots when worker_dtype == W_F32
    std::vector<std::vector<uint16_t>> th0_bf16;  // worker snapshots when worker_dtype == W_BF16
    std::vector<uint64_t> worker_round;           // arrivals seen from each worker
    std::vector<uint64_t> worker_sched_t;         // LPS counter t when the worker was last scheduled

    // Alg. 1 lines 6-7: every model starts as Theta_0, every worker is scheduled Theta_0.
    Oracle(const Config& c, const float* theta_init) : cfg(c) {
        if (c.P == 0 || c.n_lps == 0 || c.n_workers == 0 || c.worker_lps.size() != c.n_workers)
            throw std::invalid_argument("bad config");
        for (uint32_t w = 0; w < c.n_workers; ++w)
            if (c.worker_lps[w] >= c.n_lps) throw std::invalid_argument("worker_lps out of range");
        const uint64_t P = c.P;
        Theta.resize(P);
        Mg.assign(P, T(0));
        acc_g.assign(P, T(0));
        if (c.delay_l == 0 || c.delay_g == 0) throw std::invalid_argument("delay must be >= 1");
        for (uint64_t j = 0; j < P; ++j) Theta[j] = (T)theta_init[j];
        lps.resize(c.n_lps);
        for (auto& s : lps) {
            s.th = Theta;
            s.anchor = Theta;
            s.ml.assign(P, T(0));
            s.outbox.assign(P, T(0));
            s.inbox.assign(P, T(0));
            s.last_delta.assign(P, T(0));
            s.acc.assign(P, T(0));
        }
        worker_round.assign(c.n_workers, 0);
        worker_sched_t.assign(c.n_workers, 0);
        if (c.worker_dtype == W_F32) {
            th0_f32.resize(c.n_workers);
            for (auto& v : th0_f32) v.assign(theta_init, theta_init + P);
        } else {
            th0_bf16.resize(c.n_workers);
            for (auto& v : th0_bf16) {
                v.resize(P);
                for (uint64_t j = 0; j < P; ++j) v[j] = f32_to_bf16_rne(theta_init[j]);
            }
        }
    }

    // The ModelUpdate of Appendix E applied to one element with a displacement d.
    static inline void model_update(T& theta, T& m, T d, T eta, T beta, T one_minus_beta) {
        T m_new = std::fma(beta, m, d);                    // m' = beta m + d
        T u = std::fma(beta, m_new, one_minus_beta * d);   // (1-beta) d + beta m'
        theta = std::fma(eta, u, theta);                   // theta' = theta + eta u
        m = m_new;
    }

    // Delayed Nesterov step on one element with displacement d (see the header for the reading).
    static inline void delayed_nesterov(T& theta, T& m, T& acc, T d, T eps, T beta, T inv_delay, T eps_over_delay,
                                        bool refresh) {
        acc = acc + d;
        if (!refresh) {
            theta = std::fma(eps_over_delay, d, theta);        // theta' = theta + (eps/d) d
        } else {
            T m_new = std::fma(beta, m, acc * inv_delay);      // m' = beta m + acc/d
            T u = std::fma(beta, m_new, d * inv_delay);        // beta m' + d/d
            theta = std::fma(eps, u, theta);
            m = m_new;
            acc = T(0);
        }
    }

    // One server-side optimizer step of the configured kind on element (theta, m, acc).
    inline void step(T& theta, T& m, T& acc, T d, T eta, T beta, T omb, T inv_delay, T eta_over_delay, bool refresh) const {
        if (cfg.optimizer == OPT_PAPER) model_update(theta, m, d, eta, beta, omb);
        else delayed_nesterov(theta, m, acc, d, eta, beta, inv_delay, eta_over_delay, refresh);
    }

    // A worker's result theta_{t,H} reaches its LPS (Alg. 1 lines 9-15 and 25).
    // thetaH is in the worker dtype (float, or uint16_t bf16 patterns).  Returns true if the
    // arrival completed a window of K updates, in which case Delta was formed (line 14).
    bool arrive(uint32_t w, const void* thetaH) {
        if (w >= cfg.n_workers) throw std::invalid_argument("worker out of range");
        Lps<T>& s = lps[cfg.worker_lps[w]];
        const T eta = (T)cfg.eta_l, beta = (T)cfg.beta_l, omb = T(1) - beta;
        const T inv_delay = T(1) / (T)cfg.delay_l, eta_over_delay = eta * inv_delay;
        const bool refresh = ((s.t + 1) % cfg.delay_l) == 0;   // this is the LPS's update number t+1
        const uint64_t P = cfg.P;
        if (cfg.worker_dtype == W_F32) {
            const float* h = (const float*)thetaH;
            float* s0 = th0_f32[w].data();
            for (uint64_t j = 0; j < P; ++j) {
                T d = (T)h[j] - (T)s0[j];                  // line 25: delta = theta_{t,H} - theta_{t,0}
                s.last_delta[j] = d;
                step(s.th[j], s.ml[j], s.acc[j], d, eta, beta, omb, inv_delay, eta_over_delay, refresh);   // line 11
                s0[j] = (float)s.th[j];                    // line 12: schedule the worker theta_t
            }
        } else {
            const uint16_t* h = (const uint16_t*)thetaH;
            uint16_t* s0 = th0_bf16[w].data();
            for (uint64_t j = 0; j < P; ++j) {
                T d = (T)bf16_to_f32(h[j]) - (T)bf16_to_f32(s0[j]);
                s.last_delta[j] = d;
                step(s.th[j], s.ml[j], s.acc[j], d, eta, beta, omb, inv_delay, eta_over_delay, refresh);
                s0[j] = f32_to_bf16_rne((float)s.th[j]);
            }
        }
        s.t += 1;                                          // line 10
        worker_round[w] += 1;
        worker_sched_t[w] = s.t;
        if (s.t - s.t_last == cfg.K) {                     // line 13 (equality)
            push(cfg.worker_lps[w]);
            return true;
        }
        return false;
    }

    // Alg. 1 line 14: Delta = theta_t - theta_{t_last}, left in the outbox.
    void push(uint32_t l) {
        Lps<T>& s = lps.at(l);
        if (s.phase != IDLE) throw std::logic_error("push while a round trip is in flight");
        for (uint64_t j = 0; j < cfg.P; ++j) s.outbox[j] = s.th[j] - s.anchor[j];
        s.phase = PUSHED;
        s.t_push = s.t;
    }

    // Alg. 1 lines 2-4: the GPS receives the Delta of LPS l, updates Theta with global
    // momentum, and sends that Theta_i back (a snapshot: later GPS iterations do not alter it).
    void gps_recv(uint32_t l) {
        Lps<T>& s = lps.at(l);
        if (s.phase != PUSHED) throw std::logic_error("gps_recv without a pushed Delta");
        const T eta = (T)cfg.eta_g, beta = (T)cfg.beta_g, omb = T(1) - beta;
        const T inv_delay = T(1) / (T)cfg.delay_g, eta_over_delay = eta * inv_delay;
        const bool refresh = ((i + 1) % cfg.delay_g) == 0;
        for (uint64_t j = 0; j < cfg.P; ++j) {
            step(Theta[j], Mg[j], acc_g[j], s.outbox[j], eta, beta, omb, inv_delay, eta_over_delay, refresh);
            s.inbox[j] = Theta[j];
        }
        i += 1;
        s.phase = ANSWERED;
    }

    // Alg. 1 lines 17-20: merge the received Theta_i; the merged model is the new anchor.
    void pull(uint32_t l) {
        Lps<T>& s = lps.at(l);
        if (s.phase != ANSWERED) throw std::logic_error("pull without an answer from the GPS");
        const T a = (T)cfg.alpha, oma = T(1) - a;
        s.t_last = s.t;                                    // line 18
        for (uint64_t j = 0; j < cfg.P; ++j) {
            T x = std::fma(a, s.inbox[j], oma * s.th[j]);  // line 19
            s.th[j] = x;
            s.anchor[j] = x;
        }
        s.phase = IDLE;
    }
};

}  // namespace halos_oracle

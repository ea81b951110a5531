"""A second, independent reading of Algorithm 1 used only to pin the oracle.

It keeps the paper's own indexing: every LPS stores its whole model history theta[t], the GPS
stores Theta[i], and "theta_{t_last}" is looked up from that history.  ModelUpdate is written
in the gradient form of Appendix E (g = -displacement, theta' = theta - eta[(1-beta)g + beta m']).
Numbers are whatever type the caller supplies (fractions.Fraction for exact expansion, float
for double precision), one Python scalar at a time -- slow on purpose.
"""
from __future__ import annotations


class PaperInterpreter:
    def __init__(self, Theta0, worker_lps, eta_l, beta_l, eta_g, beta_g, alpha, K, zero=0):
        self.P = len(Theta0)
        self.worker_lps = list(worker_lps)
        n_lps = max(worker_lps) + 1
        self.eta_l, self.beta_l, self.eta_g, self.beta_g, self.alpha, self.K = eta_l, beta_l, eta_g, beta_g, alpha, K
        self.zero = zero
        # GPS
        self.Theta = [list(Theta0)]               # Theta[i]
        self.m_g = [zero] * self.P
        # LPS
        self.theta = [{0: list(Theta0)} for _ in range(n_lps)]   # theta[l][t]
        self.m_l = [[zero] * self.P for _ in range(n_lps)]
        self.t = [0] * n_lps
        self.t_last = [0] * n_lps
        self.delta_in_flight = [None] * n_lps     # Delta travelling to the GPS
        self.Theta_in_flight = [None] * n_lps     # Theta_i travelling back
        # workers: the model each was last scheduled with (lines 7 and 12)
        self.start = [list(Theta0) for _ in worker_lps]

    @staticmethod
    def _model_update(theta, m, displacement, eta, beta):
        new_theta, new_m = [], []
        for th, mm, d in zip(theta, m, displacement):
            g = -d
            m1 = beta * mm + g
            new_m.append(m1)
            new_theta.append(th - eta * ((1 - beta) * g + beta * m1))
        return new_theta, new_m

    def arrive(self, w, thetaH):
        l = self.worker_lps[w]
        delta = [h - s for h, s in zip(thetaH, self.start[w])]           # line 25
        self.t[l] += 1                                                   # line 10
        t = self.t[l]
        prev = self.theta[l][t - 1]
        self.theta[l][t], self.m_l[l] = self._model_update(prev, self.m_l[l], delta, self.eta_l, self.beta_l)  # 11
        self.start[w] = list(self.theta[l][t])                           # line 12
        if t - self.t_last[l] == self.K:                                 # line 13
            assert self.delta_in_flight[l] is None and self.Theta_in_flight[l] is None
            ref = self.theta[l][self.t_last[l]]
            self.delta_in_flight[l] = [a - b for a, b in zip(self.theta[l][t], ref)]   # line 14
            return True
        return False

    def gps_recv(self, l):
        Delta = self.delta_in_flight[l]
        assert Delta is not None
        self.delta_in_flight[l] = None
        new_Theta, self.m_g = self._model_update(self.Theta[-1], self.m_g, Delta, self.eta_g, self.beta_g)  # line 3
        self.Theta.append(new_Theta)
        self.Theta_in_flight[l] = list(new_Theta)                        # line 4

    def pull(self, l):
        Th = self.Theta_in_flight[l]
        assert Th is not None
        self.Theta_in_flight[l] = None
        t = self.t[l]
        self.t_last[l] = t                                               # line 18
        a = self.alpha
        self.theta[l][t] = [(1 - a) * x + a * y for x, y in zip(self.theta[l][t], Th)]   # line 19

    # convenience
    def lps_model(self, l):
        return self.theta[l][self.t[l]]

    def gps_model(self):
        return self.Theta[-1]

"""Sequence-aware trigger: which requests get a pre-infer, and how many (paper Section 3.2).

Host arithmetic only.  The trigger looks at metadata (the prefix length), skips users whose full inference is not
at risk, and admits the rest while two budgets hold: the live caches of one lifecycle window must fit the share of
HBM reserved for them (Eq. 1, 2), and the admitted rate must stay within what the instance's model slots sustain
(Eq. 3).  ``from_measurements`` fills the budgets from numbers this library reports: the K/V bytes of a prefix
(``relaygr_kv_page_bytes``) and a measured pre-infer time.
"""
from __future__ import annotations

import math
from collections import deque
from dataclasses import dataclass


@dataclass(frozen=True)
class AdmissionLimits:
    live_caches: int            # L: caches alive at once in one special instance (Eq. 2)
    admit_qps_compute: float    # Q_m * M (Eq. 3, first inequality)
    admit_qps_survival: float   # L / T_life (Eq. 1)
    pool_qps: float             # (Q_m * M) * (r2 * N) (Eq. 3, second inequality)

    @property
    def admit_qps(self) -> float:
        return min(self.admit_qps_compute, self.admit_qps_survival)


def limits(q_m: float, n_slots: int, kv_p99_bytes: float, hbm_bytes: float, r1: float, t_life_s: float, r2: float = 1.0,
           n_instances: int = 1) -> AdmissionLimits:
    live = int(math.floor(r1 * hbm_bytes / kv_p99_bytes + 1e-9))
    per_instance = q_m * n_slots
    return AdmissionLimits(live, per_instance, live / t_life_s, per_instance * r2 * n_instances)


def from_measurements(preinfer_ms: float, kv_bytes_per_user: int, hbm_bytes: int, r1: float, t_life_s: float, n_slots: int = 1,
                      r2: float = 1.0, n_instances: int = 1) -> AdmissionLimits:
    """Budgets from a measured pre-infer latency (ms per user, one slot) and the pool's K/V footprint per user."""
    return limits(1000.0 / preinfer_ms, n_slots, float(kv_bytes_per_user), float(hbm_bytes), r1, t_life_s, r2, n_instances)


class Trigger:
    """Admits at-risk requests while the budgets hold.  ``risk_threshold`` is the prefix length from which full
    inference endangers the ranking-stage P99 (the paper's special-instance threshold, e.g. 4K tokens)."""

    def __init__(self, lim: AdmissionLimits, risk_threshold: int, t_life_s: float):
        self.lim, self.risk_threshold, self.t_life_s = lim, int(risk_threshold), float(t_life_s)
        self._live = deque()            # admission times of caches still inside their lifecycle window
        self._recent = deque()          # admission times within the last second
        self.skipped = self.admitted = self.rejected = 0

    def offer(self, now_s: float, prefix_len: int) -> bool:
        """True = send the pre-infer signal for this user; False = leave the request to ordinary inference."""
        if prefix_len < self.risk_threshold:
            self.skipped += 1                                   # not at risk: zero extra work
            return False
        while self._live and now_s - self._live[0] >= self.t_life_s:
            self._live.popleft()
        while self._recent and now_s - self._recent[0] >= 1.0:
            self._recent.popleft()
        if len(self._live) >= self.lim.live_caches or len(self._recent) + 1 > self.lim.admit_qps_compute:
            self.rejected += 1
            return False
        self._live.append(now_s)
        self._recent.append(now_s)
        self.admitted += 1
        return True

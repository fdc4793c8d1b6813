"""Plain restatement of the sequence-aware trigger's admission bounds (paper Section 3.2, Eq. 1-3).

TEST INFRASTRUCTURE ONLY, like the rest of ``oracle/``: nothing on the product path imports it, and it imports
nothing from the product.

    Eq. 1   L = Q_admit * T_life                      live caches per special instance
    Eq. 2   L * kv_p99 <= r1 * HBM                    survivability in the lifecycle window
    Eq. 3   Q_admit <= Q_m * M ;  Q_max <= (Q_m * M) * (r2 * N)

Pin: the worked example of Section 3.2 (tests/golden/trigger_example.txt): 160 live caches, 150 QPS per special
instance, 1500 QPS for the pool.
"""


def max_live_caches(kv_p99_gb: float, hbm_gb: float, r1: float) -> float:
    """Largest L that Eq. 2 allows."""
    return r1 * hbm_gb / kv_p99_gb


def max_admit_rate_compute(q_m: float, n_slots: int) -> float:
    """First inequality of Eq. 3."""
    return q_m * n_slots


def max_admit_rate_survival(kv_p99_gb: float, hbm_gb: float, r1: float, t_life_s: float) -> float:
    """Eq. 1 solved for Q_admit under Eq. 2."""
    return max_live_caches(kv_p99_gb, hbm_gb, r1) / t_life_s


def max_pool_rate(q_m: float, n_slots: int, r2: float, n_instances: int) -> float:
    """Second inequality of Eq. 3."""
    return q_m * n_slots * (r2 * n_instances)

"""The sequence-aware trigger (paper Section 3.2): the plain restatement against the paper's worked example, and the
product calculator / trigger against that restatement."""
import os

import numpy as np

from oracle import admission as oracle_adm
from paper_2601_01712_b200 import admission, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _example():
    rows = [l.split() for l in open(os.path.join(ROOT, "tests", "golden", "trigger_example.txt")) if not l.startswith("#")]
    return [float(x) for x in rows[0]]


def test_restatement_reproduces_the_papers_example():
    q_m, M, kv, hbm, r1, N, r2, L, q_admit, q_max = _example()
    assert abs(oracle_adm.max_live_caches(kv, hbm, r1) - L) < 1e-9
    assert oracle_adm.max_admit_rate_compute(q_m, int(M)) == q_admit
    assert abs(oracle_adm.max_pool_rate(q_m, int(M), r2, int(N)) - q_max) < 1e-9
    # Eq. 1: the survival bound scales as 1 / T_life
    assert abs(oracle_adm.max_admit_rate_survival(kv, hbm, r1, 0.5) - 2 * L) < 1e-9


def test_calculator_matches_the_restatement():
    q_m, M, kv, hbm, r1, N, r2, L, q_admit, q_max = _example()
    lim = admission.limits(q_m, int(M), kv * 1e9, hbm * 1e9, r1, t_life_s=0.4, r2=r2, n_instances=int(N))
    assert lim.live_caches == int(L) and lim.admit_qps_compute == q_admit and abs(lim.pool_qps - q_max) < 1e-9
    assert abs(lim.admit_qps_survival - oracle_adm.max_admit_rate_survival(kv, hbm, r1, 0.4)) < 1e-9
    assert lim.admit_qps == min(q_admit, L / 0.4)
    rng = np.random.default_rng(3)
    for _ in range(50):
        q, m_, k, h, r, t = rng.uniform(1, 100), int(rng.integers(1, 9)), rng.uniform(0.01, 1), rng.uniform(8, 192), rng.uniform(0.1, 0.9), rng.uniform(0.05, 2)
        lim = admission.limits(q, m_, k, h, r, t)
        assert lim.live_caches == int(np.floor(oracle_adm.max_live_caches(k, h, r) + 1e-9))
        assert abs(lim.admit_qps_compute - oracle_adm.max_admit_rate_compute(q, m_)) < 1e-9


def test_budgets_from_this_librarys_own_numbers():
    shape = synth.MODEL_LONG                                  # 8 layers, d_model 512, bf16
    kv = shape.kv_bytes(8192)                                 # 128 MiB per user
    lim = admission.from_measurements(preinfer_ms=1.4, kv_bytes_per_user=kv, hbm_bytes=64 << 30, r1=0.5, t_life_s=0.3, n_slots=2)
    assert lim.live_caches == (32 << 30) // kv == 256
    assert abs(lim.admit_qps_compute - 2 * 1000 / 1.4) < 1e-9


def test_trigger_skips_short_users_and_respects_both_budgets():
    lim = admission.AdmissionLimits(live_caches=5, admit_qps_compute=100.0, admit_qps_survival=10.0, pool_qps=1000.0)
    trig = admission.Trigger(lim, risk_threshold=4096, t_life_s=0.5)
    assert not trig.offer(0.0, 1000) and trig.skipped == 1                 # not at risk
    got = [trig.offer(0.01 * i, 8192) for i in range(10)]                  # 10 long users within 0.1 s
    assert got == [True] * 5 + [False] * 5                                 # live-cache budget
    assert trig.offer(0.6, 8192)                                           # the window moved on
    fast = admission.Trigger(admission.AdmissionLimits(1000, 3.0, 1e9, 1e9), 1, t_life_s=0.001)
    assert [fast.offer(0.1 * i, 10) for i in range(5)] == [True, True, True, False, False]      # at most 3 per second

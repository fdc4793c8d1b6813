"""Per-user ordering in front of the pool (paper Section 3.4): single-flight reloads under a burst of ranks, fallback
without blocking when the cache is not there, arrival order per user.  CPU only: a host-only pool whose events the test
completes by hand, and stand-ins for the compute calls."""
import threading
import time

from paper_2601_01712_b200 import binding as B
from paper_2601_01712_b200 import frontend
from tests.test_boundary_cpu import HostPool


def _ctl(hp, what, arg=0):
    return B.relaygr_kv_host_backend_control(hp.pool, what, arg)[1]


def _commit(hp, user):
    return lambda: B.relaygr_kv_commit(hp.pool, user)          # stands in for relaygr_preinfer on a host-only context


def test_burst_of_ranks_for_a_spilled_user_causes_one_reload():
    hp = HostPool(4, 8)
    gate = frontend.UserGate(hp.pool)
    assert gate.preinfer(7, 128, _commit(hp, 7)) == frontend.MISS
    assert gate.evict(7, True) == frontend.HIT
    assert B.relaygr_kv_lookup(hp.pool, 7)[0] == B.TIER_HOST
    _ctl(hp, B.HOSTCTL_MANUAL_EVENTS, 1)                       # the reload stays in flight while the burst arrives
    ranked, results = [], []

    def one(i):
        results.append(gate.rank(7, lambda: ranked.append(i)))

    threads = [threading.Thread(target=one, args=(i,)) for i in range(8)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    st = B.relaygr_kv_stats(hp.pool)
    assert st["reloads"] == 1 and st["users_loading"] == 1     # the first probe reloads, the others find it on its way
    assert results == [frontend.HIT] * 8 and sorted(ranked) == list(range(8))
    assert gate.evict(7, False) == frontend.BUSY               # not while its reload is in flight
    _ctl(hp, B.HOSTCTL_COMPLETE_EVENTS, -1)
    assert gate.rank(7, lambda: None) == frontend.HIT and B.relaygr_kv_stats(hp.pool)["reloads"] == 1
    assert gate.evict(7, False) == frontend.HIT


def test_rank_before_its_preinfer_falls_back_and_never_blocks():
    hp = HostPool(4, 4)
    gate = frontend.UserGate(hp.pool)
    called = []
    t0 = time.perf_counter()
    assert gate.rank(3, lambda: called.append("rank")) == frontend.MISS       # unknown user: full inference instead
    assert time.perf_counter() - t0 < 0.5 and not called
    # the pre-infer signal arrives; a second, duplicate signal is harmless
    assert gate.preinfer(3, 64, _commit(hp, 3)) == frontend.MISS
    assert gate.preinfer(3, 64, lambda: called.append("again")) == frontend.HIT and not called
    assert gate.rank(3, lambda: called.append("rank")) == frontend.HIT and called == ["rank"]
    # evicted without a DRAM copy: a miss again
    assert gate.evict(3, False) == frontend.HIT
    assert gate.rank(3, lambda: called.append("rank")) == frontend.MISS and called == ["rank"]
    # a user whose pages are reserved but whose pre-infer has not been enqueued is a miss too
    B.relaygr_kv_alloc(hp.pool, 4, 64)
    assert gate.rank(4, lambda: called.append("rank4")) == frontend.MISS and "rank4" not in called
    # no room: the signal is refused, nothing waits
    assert gate.preinfer(5, 64 * 10, lambda: None) == frontend.BUSY


def test_requests_of_one_user_run_in_arrival_order():
    hp = HostPool(8, 8)
    gate = frontend.UserGate(hp.pool)
    release = threading.Event()
    order = []

    def slow_preinfer():
        release.wait(5)                                        # user 1's pre-infer is still being enqueued ...
        B.relaygr_kv_commit(hp.pool, 1)

    t1 = threading.Thread(target=lambda: order.append(("pre", gate.preinfer(1, 64, slow_preinfer))))
    t1.start()
    while not gate._next:                                      # ... its ticket is taken
        time.sleep(0.001)
    t2 = threading.Thread(target=lambda: order.append(("rank", gate.rank(1, lambda: None))))
    t2.start()                                                 # a rank of the same user queues behind it
    time.sleep(0.05)
    assert order == []
    release.set()
    t1.join(); t2.join()
    assert order == [("pre", frontend.MISS), ("rank", frontend.HIT)]          # the rank ran after the pre-infer, and hit
    assert [k for (_, k, _) in gate.log] == ["preinfer", "rank-hit"]
    assert not gate._next and not gate._serving                # nothing is kept for idle users

"""Per-user ordering in front of one prefix-KV pool (paper Section 3.4, "single-flight" and the per-user queue).

A ranking instance receives, for one user, a pre-infer signal, one or more rank requests and - from its own cache
manager - evictions; they come from different threads and may arrive in any order.  The paper serialises the operations
of one user with a per-user queue or lock, precedes every rank by an idempotent "pseudo pre-infer" that probes HBM and
then DRAM, and lets only the first of several concurrent requests trigger the reload.  A request whose cache is not
there never waits for it: it falls back to full inference (Section 3.1, invariant I1).

``UserGate`` is that front: requests of one user run one at a time, in arrival order; requests of different users do
not wait for one another beyond the library call itself (the pool's host calls must come from one thread at a time, so
each is made under one pool-wide lock).  It holds no arithmetic and moves no data: the callables it is given make the
actual ``relaygr_preinfer`` / ``relaygr_rank`` calls.
"""
from __future__ import annotations

import threading
from collections import defaultdict
from typing import Callable, Dict, Optional

from . import binding as B

HIT, MISS, BUSY = "hit", "miss", "busy"


class UserGate:
    def __init__(self, pool_handle, side_stream: Optional[int] = None):
        """pool_handle: the relaygr_kv_pool pointer; side_stream: the cudaStream_t reloads and spills are enqueued on."""
        self.pool = pool_handle
        self.side = side_stream
        self._mu = threading.Condition()            # guards the tickets
        self._lib = threading.Lock()                # one library call on the pool at a time
        self._next: Dict[int, int] = defaultdict(int)
        self._serving: Dict[int, int] = defaultdict(int)
        self.log = []                               # (user, kind, ticket) in execution order, for tests and tracing

    # ---- per-user FIFO ------------------------------------------------------------------------------------------
    def _enter(self, user: int) -> int:
        with self._mu:
            t = self._next[user]
            self._next[user] = t + 1
            while self._serving[user] != t:
                self._mu.wait()
            return t

    def _leave(self, user: int):
        with self._mu:
            self._serving[user] += 1
            if self._serving[user] == self._next[user]:        # nobody queued: forget the user
                del self._serving[user], self._next[user]
            self._mu.notify_all()

    def _probe_locked(self, user: int) -> str:
        """The pseudo pre-infer: HBM, then DRAM (one reload at most, however many requests probe)."""
        code, _ = B.relaygr_kv_reload_from_host(self.pool, user, self.side, ok=(B.OK, B.E_MISS, B.E_BUSY, B.E_NOSPACE))
        if code == B.OK:
            return HIT                      # resident, loading (single-flight), or the reload has just been enqueued
        return MISS if code == B.E_MISS else BUSY       # E_BUSY: too many reloads in flight; E_NOSPACE: the window is full

    # ---- requests -------------------------------------------------------------------------------------------------
    def preinfer(self, user: int, prefix_len: int, run: Callable[[], None]) -> str:
        """A pre-infer signal.  A user that already has a cache in any tier is left alone (duplicate signals are
        harmless); else pages are reserved and ``run()`` makes the relaygr_preinfer call.  Returns HIT if a cache
        existed, BUSY if the pool had no room (the caller's window policy decides what to evict), else MISS -> computed."""
        t = self._enter(user)
        try:
            with self._lib:
                tier, _ = B.relaygr_kv_lookup(self.pool, user)
                if tier != B.TIER_MISS:
                    self.log.append((user, "preinfer-duplicate", t))
                    return HIT
                if B.relaygr_kv_alloc(self.pool, user, prefix_len, ok=(B.OK, B.E_NOSPACE)) != B.OK:
                    self.log.append((user, "preinfer-nospace", t))
                    return BUSY
                run()
            self.log.append((user, "preinfer", t))
            return MISS
        finally:
            self._leave(user)

    def rank(self, user: int, run: Callable[[], None]) -> str:
        """A rank request: probe first; ``run()`` (the relaygr_rank call) only if the user's cache is in HBM or on its
        way there.  MISS / BUSY return at once - the caller ranks by full inference."""
        t = self._enter(user)
        try:
            with self._lib:
                state = self._probe_locked(user)
                if state == HIT:
                    tier, _ = B.relaygr_kv_lookup(self.pool, user)
                    if tier == B.TIER_ALLOCATED:        # reserved, its pre-infer not enqueued yet: nothing to rank on
                        state = MISS
                if state == HIT:
                    run()
            self.log.append((user, "rank-" + state, t))
            return state
        finally:
            self._leave(user)

    def evict(self, user: int, spill_to_host: bool) -> str:
        """An eviction by the cache manager.  BUSY while the user's reload is in flight (it is not waited for)."""
        t = self._enter(user)
        try:
            with self._lib:
                code = B.relaygr_kv_evict(self.pool, user, spill_to_host, self.side, ok=(B.OK, B.E_MISS, B.E_BUSY, B.E_NOSPACE))
            state = HIT if code == B.OK else (MISS if code == B.E_MISS else BUSY)
            self.log.append((user, "evict-" + state, t))
            return state
        finally:
            self._leave(user)

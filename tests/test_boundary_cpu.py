"""CPU-only checks of the boundary: the library loads, exports every symbol the header
declares, refuses to compute without a device, and the pool's host logic (state machine,
page accounting, single-flight reload, spill / reload byte-exactness) behaves as the
header says.  Uses the host-only context: tiers are plain host memory."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2601_01712_b200 import binding as B
from paper_2601_01712_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()


def test_every_declared_symbol_is_exported_and_bound():
    hdr = open(os.path.join(ROOT, "include", "relaygr.h")).read()
    declared = set(re.findall(r"^(?:int32_t|const char \*)\s*(relaygr_[a-z0-9_]+)\s*\(", hdr, flags=re.M))
    assert len(declared) >= 20
    lib = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), "missing export: " + name
    assert declared == set(B.SIGNATURES), declared ^ set(B.SIGNATURES)


def _cfg(dtype=B.DTYPE_BF16, L=2, d=128, H=2, F=256):
    return B.ModelCfg(L, d, H, d // H, F, dtype, 64, 1000, 1e-5)


def test_shape_validation():
    for bad in (B.ModelCfg(2, 128, 2, 32, 256, B.DTYPE_BF16, 64, 10, 1e-5),      # bf16 needs d_head 64
                B.ModelCfg(2, 128, 2, 64, 256, B.DTYPE_BF16, 32, 10, 1e-5),      # page size
                B.ModelCfg(2, 100, 2, 64, 256, B.DTYPE_F32, 64, 10, 1e-5),       # heads * d_head != d
                B.ModelCfg(0, 128, 2, 64, 256, B.DTYPE_F32, 64, 10, 1e-5)):
        with pytest.raises(B.RelayGRError):
            B.relaygr_create_host_only(bad)
    assert "d_head" in B.last_error() or "n_layers" in B.last_error() or "positive" in B.last_error()
    with pytest.raises(B.RelayGRError):                                          # attn_kind is softmax (0) or pointwise (1)
        B.relaygr_create_host_only(B.ModelCfg(2, 128, 2, 64, 256, B.DTYPE_F32, 64, 10, 1e-5, 2))
    assert "attn_kind" in B.last_error()


def test_both_attention_kinds_are_accepted():
    for kind in (0, 1):
        ctx = B.relaygr_create_host_only(B.ModelCfg(2, 128, 2, 64, 256, B.DTYPE_BF16, 64, 10, 1e-5, kind))
        B.relaygr_destroy(ctx)


def test_no_cpu_compute_path():
    ctx = B.relaygr_create_host_only(_cfg())
    slab = np.zeros(4 * B.relaygr_kv_page_bytes(ctx) + 1024, dtype=np.uint8)
    base = (slab.ctypes.data + 1023) // 1024 * 1024
    pool = B.relaygr_kv_pool_create(ctx, base, 4 * B.relaygr_kv_page_bytes(ctx))
    B.relaygr_kv_alloc(pool, 1, 64)
    off = np.array([0, 64], np.int32)
    with pytest.raises(B.RelayGRError) as e:
        B.relaygr_preinfer(ctx, pool, [1], 0x1000, off)
    assert e.value.code == B.E_UNSUPPORTED
    with pytest.raises(B.RelayGRError) as e:
        B.relaygr_rank_full(ctx, 1, 0x1000, off, 0x1000, off, 0x1000, off, 0x1000)
    assert e.value.code == B.E_UNSUPPORTED
    with pytest.raises(B.RelayGRError):
        B.relaygr_gather(ctx, 0x1000, 4, 0x1000)
    B.relaygr_kv_pool_destroy(pool)
    B.relaygr_destroy(ctx)


class HostPool:
    def __init__(self, hbm_pages, host_pages, cfg=None):
        self.ctx = B.relaygr_create_host_only(cfg or _cfg())
        self.pb = B.relaygr_kv_page_bytes(self.ctx)
        self._hbm = np.zeros(hbm_pages * self.pb + 1024, dtype=np.uint8)
        off = (-self._hbm.ctypes.data) % 1024
        self.hbm = self._hbm[off:off + hbm_pages * self.pb]
        self.host = np.zeros(max(1, host_pages * self.pb), dtype=np.uint8)
        self.pool = B.relaygr_kv_pool_create(self.ctx, self.hbm.ctypes.data, hbm_pages * self.pb,
                                             self.host.ctypes.data if host_pages else None, host_pages * self.pb)

    def page(self, i):
        return self.hbm[i * self.pb:(i + 1) * self.pb]


def test_page_bytes_and_accounting():
    hp = HostPool(10, 0)
    assert hp.pb == 2 * 2 * 64 * 128 * 2
    st = B.relaygr_kv_stats(hp.pool)
    assert st["pages_total"] == 10 and st["pages_free"] == 10
    B.relaygr_kv_alloc(hp.pool, 5, 65)                  # 2 pages
    B.relaygr_kv_alloc(hp.pool, 6, 64 * 3)              # 3 pages
    assert list(B.relaygr_kv_pages(hp.pool, 5)) == [0, 1]
    assert list(B.relaygr_kv_pages(hp.pool, 6)) == [2, 3, 4]
    assert B.relaygr_kv_stats(hp.pool)["pages_free"] == 5
    assert B.relaygr_kv_alloc(hp.pool, 5, 10, ok=(B.E_EXISTS,)) == B.E_EXISTS
    assert B.relaygr_kv_alloc(hp.pool, 7, 64 * 6, ok=(B.E_NOSPACE,)) == B.E_NOSPACE
    assert B.relaygr_kv_stats(hp.pool)["pages_free"] == 5          # a failed alloc takes nothing
    assert B.relaygr_kv_alloc(hp.pool, 7, 0, ok=(B.E_INVALID,)) == B.E_INVALID
    assert B.relaygr_kv_lookup(hp.pool, 5) == (B.TIER_ALLOCATED, 65)
    assert B.relaygr_kv_lookup(hp.pool, 99) == (B.TIER_MISS, 0)
    B.relaygr_kv_free(hp.pool, 5)
    assert B.relaygr_kv_free(hp.pool, 5, ok=(B.E_MISS,)) == B.E_MISS
    assert B.relaygr_kv_stats(hp.pool)["pages_free"] == 7
    # caller-chosen (shuffled) pages
    B.relaygr_kv_alloc(hp.pool, 8, 64 * 3, [9, 0, 7])
    assert list(B.relaygr_kv_pages(hp.pool, 8)) == [9, 0, 7]
    assert B.relaygr_kv_alloc(hp.pool, 9, 64, [9], ok=(B.E_NOSPACE,)) == B.E_NOSPACE     # in use
    assert B.relaygr_kv_alloc(hp.pool, 9, 64, [10], ok=(B.E_INVALID,)) == B.E_INVALID    # out of range
    assert B.relaygr_kv_alloc(hp.pool, 9, 128, [5, 5], ok=(B.E_NOSPACE,)) == B.E_NOSPACE  # repeated
    # everything that is free can still be handed out exactly once
    B.relaygr_kv_alloc(hp.pool, 10, 64 * 4)
    got = set(B.relaygr_kv_pages(hp.pool, 10))
    assert len(got) == 4 and not (got & {9, 0, 7, 2, 3, 4})
    assert B.relaygr_kv_stats(hp.pool)["pages_free"] == 0
    assert B.relaygr_kv_alloc(hp.pool, 11, 1, ok=(B.E_NOSPACE,)) == B.E_NOSPACE


def _make_resident(hp, user, prefix_len, fill):
    """Host-only stand-in for pre-infer: there is no compute, so write a byte pattern into the
    user's pages (each page gets fill + its logical index) and leave the entry ALLOCATED."""
    B.relaygr_kv_alloc(hp.pool, user, prefix_len)
    for i, p in enumerate(B.relaygr_kv_pages(hp.pool, user)):
        hp.page(p)[:] = (fill + i) % 251


def test_evict_of_allocated_entry_and_host_states():
    hp = HostPool(6, 6)
    _make_resident(hp, 1, 128, 11)
    # ALLOCATED entries hold no content: evict just returns the pages and drops the entry
    B.relaygr_kv_evict(hp.pool, 1, 1)
    assert B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_MISS
    assert B.relaygr_kv_stats(hp.pool)["pages_free"] == 6
    code, ev = B.relaygr_kv_reload_from_host(hp.pool, 1, ok=(B.E_MISS,))
    assert code == B.E_MISS and ev is None
    _make_resident(hp, 2, 64, 3)
    code, _ = B.relaygr_kv_reload_from_host(hp.pool, 2, ok=(B.E_MISS,))     # never pre-inferred
    assert code == B.E_MISS
    assert B.relaygr_kv_evict(hp.pool, 42, 1, ok=(B.E_MISS,)) == B.E_MISS


def test_many_alloc_free_cycles_keep_the_free_list_exact():
    hp = HostPool(8, 0)
    rng = np.random.default_rng(0)
    live = {}
    for step in range(400):
        u = int(rng.integers(0, 12))
        if u in live:
            B.relaygr_kv_free(hp.pool, u)
            del live[u]
        else:
            n = int(rng.integers(1, 4))
            free = B.relaygr_kv_stats(hp.pool)["pages_free"]
            ids = None
            if step % 3 == 0:
                used = set(int(p) for v in live.values() for p in v)
                cand = [p for p in range(8) if p not in used]
                ids = list(rng.permutation(cand)[:n]) if len(cand) >= n else None
            code = B.relaygr_kv_alloc(hp.pool, u, n * 64, ids, ok=(B.OK, B.E_NOSPACE))
            assert (code == B.OK) == (free >= n)
            if code == B.OK:
                live[u] = list(B.relaygr_kv_pages(hp.pool, u))
        pages = [p for v in live.values() for p in v]
        assert len(pages) == len(set(pages))
        assert B.relaygr_kv_stats(hp.pool)["pages_free"] == 8 - len(pages)


def _content(hp, user):
    return [hp.page(p).copy() for p in B.relaygr_kv_pages(hp.pool, user)]


def test_spill_reload_state_machine_single_flight_and_bytes():
    """Section 3.4: two-level lookup, spill after use, reload at most once, bytes preserved."""
    hp = HostPool(4, 8)
    _make_resident(hp, 1, 128, 10)
    assert B.relaygr_kv_commit(hp.pool, 99, ok=(B.E_MISS,)) == B.E_MISS
    B.relaygr_kv_commit(hp.pool, 1)
    assert B.relaygr_kv_commit(hp.pool, 1, ok=(B.E_INVALID,)) == B.E_INVALID
    assert B.relaygr_kv_lookup(hp.pool, 1) == (B.TIER_HBM, 128)
    want = _content(hp, 1)
    # resident: reload is a no-op
    assert B.relaygr_kv_reload_from_host(hp.pool, 1) == (B.OK, None)
    assert B.relaygr_kv_stats(hp.pool)["reloads"] == 0
    # spill, then fill HBM with other users
    B.relaygr_kv_evict(hp.pool, 1, 1)
    assert B.relaygr_kv_lookup(hp.pool, 1) == (B.TIER_HOST, 128)
    assert B.relaygr_kv_evict(hp.pool, 1, 1, ok=(B.E_MISS,)) == B.E_MISS            # holds no HBM pages now
    st = B.relaygr_kv_stats(hp.pool)
    assert st["pages_free"] == 4 and st["host_pages_free"] == 6 and st["spills"] == 1 and st["spill_bytes"] == 2 * hp.pb
    _make_resident(hp, 2, 256, 77)
    B.relaygr_kv_commit(hp.pool, 2)
    code, _ = B.relaygr_kv_reload_from_host(hp.pool, 1, ok=(B.E_NOSPACE,))
    assert code == B.E_NOSPACE and B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_HOST
    # evict user 2 without spilling: dropped entirely
    B.relaygr_kv_evict(hp.pool, 2, 0)
    assert B.relaygr_kv_lookup(hp.pool, 2)[0] == B.TIER_MISS
    hp.hbm[:] = 0xEE
    # first probe reloads, later probes find it in HBM (pseudo pre-infer before every rank)
    for _ in range(3):
        code, _ = B.relaygr_kv_reload_from_host(hp.pool, 1)
        assert code == B.OK
    st = B.relaygr_kv_stats(hp.pool)
    assert st["reloads"] == 1 and st["reload_bytes"] == 2 * hp.pb
    assert B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_HBM
    got = _content(hp, 1)
    assert all(np.array_equal(a, b) for a, b in zip(got, want))
    # the host copy is kept: the next eviction needs no second spill copy
    B.relaygr_kv_evict(hp.pool, 1, 1)
    assert B.relaygr_kv_stats(hp.pool)["spills"] == 1
    assert B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_HOST
    # evict without spill while a host copy exists keeps the entry in the host tier
    B.relaygr_kv_reload_from_host(hp.pool, 1)
    B.relaygr_kv_evict(hp.pool, 1, 0)
    assert B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_HOST
    B.relaygr_kv_free(hp.pool, 1)
    st = B.relaygr_kv_stats(hp.pool)
    assert st["host_pages_free"] == 8 and st["pages_free"] == 4 and st["users_host"] == 0


def test_host_tier_full_and_absent():
    hp = HostPool(4, 1)
    _make_resident(hp, 1, 128, 1)
    B.relaygr_kv_commit(hp.pool, 1)
    assert B.relaygr_kv_evict(hp.pool, 1, 1, ok=(B.E_NOSPACE,)) == B.E_NOSPACE       # 2 pages do not fit in 1
    assert B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_HBM                          # nothing changed
    hp2 = HostPool(4, 0)
    _make_resident(hp2, 1, 64, 1)
    B.relaygr_kv_commit(hp2.pool, 1)
    assert B.relaygr_kv_evict(hp2.pool, 1, 1, ok=(B.E_NOSPACE,)) == B.E_NOSPACE


def test_lookup_counts_hits_by_tier():
    hp = HostPool(4, 4)
    _make_resident(hp, 1, 64, 1)
    B.relaygr_kv_commit(hp.pool, 1)
    B.relaygr_kv_lookup(hp.pool, 1)
    B.relaygr_kv_lookup(hp.pool, 2)
    B.relaygr_kv_evict(hp.pool, 1, 1)
    B.relaygr_kv_lookup(hp.pool, 1)
    st = B.relaygr_kv_stats(hp.pool)
    assert (st["hits_hbm"], st["hits_host"], st["misses"]) == (1, 1, 1)


# ---------------------------------------------------------------- states that need time on a GPU (Section 3.4), held by hand
def _ctl(hp, what, arg=0):
    return B.relaygr_kv_host_backend_control(hp.pool, what, arg)[1]


def _resident(hp, user, prefix_len, fill):
    _make_resident(hp, user, prefix_len, fill)
    B.relaygr_kv_commit(hp.pool, user)


def test_loading_state_busy_codes_and_promotion():
    """A reload in flight: LOADING, single-flight, E_BUSY on evict / free, HBM once its event completes."""
    hp = HostPool(4, 8)
    _resident(hp, 1, 128, 5)
    want = _content(hp, 1)
    B.relaygr_kv_evict(hp.pool, 1, 1)
    hp.hbm[:] = 0
    _ctl(hp, B.HOSTCTL_MANUAL_EVENTS, 1)
    code, ev = B.relaygr_kv_reload_from_host(hp.pool, 1)
    assert code == B.OK and ev is not None
    assert B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_LOADING
    code2, ev2 = B.relaygr_kv_reload_from_host(hp.pool, 1)          # single-flight: the same event, nothing new enqueued
    assert code2 == B.OK and ev2 == ev and B.relaygr_kv_stats(hp.pool)["reloads"] == 1
    assert B.relaygr_kv_evict(hp.pool, 1, 1, ok=(B.E_BUSY,)) == B.E_BUSY
    assert B.relaygr_kv_evict(hp.pool, 1, 0, ok=(B.E_BUSY,)) == B.E_BUSY
    assert B.relaygr_kv_free(hp.pool, 1, ok=(B.E_BUSY,)) == B.E_BUSY
    st = B.relaygr_kv_stats(hp.pool)
    assert st["users_loading"] == 1 and st["users_hbm"] == 0
    assert _ctl(hp, B.HOSTCTL_COMPLETE_EVENTS, -1) >= 1
    assert B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_HBM
    assert B.relaygr_kv_reload_from_host(hp.pool, 1) == (B.OK, None)
    assert all(np.array_equal(a, b) for a, b in zip(_content(hp, 1), want))
    B.relaygr_kv_evict(hp.pool, 1, 0)                                # allowed again
    assert B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_HOST


def test_bounded_number_of_reloads_in_flight():
    """Section 3.4: reloads are rate-limited; beyond the bound the probe reports E_BUSY and the user stays in DRAM."""
    hp = HostPool(8, 8)
    for u in (1, 2, 3):
        _resident(hp, u, 64, u)
        B.relaygr_kv_evict(hp.pool, u, 1)
    B.relaygr_kv_set_max_inflight_reloads(hp.pool, 2)
    _ctl(hp, B.HOSTCTL_MANUAL_EVENTS, 1)
    assert B.relaygr_kv_reload_from_host(hp.pool, 1)[0] == B.OK
    assert B.relaygr_kv_reload_from_host(hp.pool, 2)[0] == B.OK
    code, ev = B.relaygr_kv_reload_from_host(hp.pool, 3, ok=(B.E_BUSY,))
    assert code == B.E_BUSY and ev is None
    assert B.relaygr_kv_lookup(hp.pool, 3)[0] == B.TIER_HOST
    assert B.relaygr_kv_stats(hp.pool)["pages_free"] == 6            # the refused reload took no pages
    assert _ctl(hp, B.HOSTCTL_COMPLETE_EVENTS, 1) == 1               # the oldest reload lands
    assert B.relaygr_kv_reload_from_host(hp.pool, 3)[0] == B.OK
    assert B.relaygr_kv_stats(hp.pool)["reloads"] == 3


def test_failed_reload_leaves_the_user_in_dram_with_its_pages_returned():
    hp = HostPool(4, 8)
    _resident(hp, 1, 128, 9)
    want = _content(hp, 1)
    B.relaygr_kv_evict(hp.pool, 1, 1)
    _ctl(hp, B.HOSTCTL_FAIL_COPIES, 1)
    code, ev = B.relaygr_kv_reload_from_host(hp.pool, 1, ok=(B.E_CUDA,))
    assert code == B.E_CUDA and ev is None
    assert B.relaygr_kv_lookup(hp.pool, 1) == (B.TIER_HOST, 128)
    st = B.relaygr_kv_stats(hp.pool)
    assert st["pages_free"] == 4 and st["reloads"] == 0 and st["host_pages_free"] == 6
    hp.hbm[:] = 0
    assert B.relaygr_kv_reload_from_host(hp.pool, 1)[0] == B.OK      # the next probe succeeds
    assert all(np.array_equal(a, b) for a, b in zip(_content(hp, 1), want))


def test_failed_spill_changes_nothing():
    hp = HostPool(4, 8)
    _resident(hp, 1, 128, 9)
    _ctl(hp, B.HOSTCTL_FAIL_COPIES, 1)
    assert B.relaygr_kv_evict(hp.pool, 1, 1, ok=(B.E_CUDA,)) == B.E_CUDA
    assert B.relaygr_kv_lookup(hp.pool, 1)[0] == B.TIER_HBM
    st = B.relaygr_kv_stats(hp.pool)
    assert st["host_pages_free"] == 8 and st["pages_free"] == 2 and st["spills"] == 0


def test_pages_stay_behind_an_earlier_owners_spill_when_they_change_hands_twice():
    """User A's spill copy is still running when its pages go to B, who gives them back without using them; the next
    owner must still wait for A's copy (a page remembers every pending ticket, not only the last owner's)."""
    hp = HostPool(2, 8)
    _resident(hp, 1, 64, 1)                                          # A: page 0
    _resident(hp, 3, 64, 3)                                          # C: page 1
    B.relaygr_kv_evict(hp.pool, 3, 1)                                # C's spill completes at once
    _ctl(hp, B.HOSTCTL_MANUAL_EVENTS, 1)
    B.relaygr_kv_evict(hp.pool, 1, 1)                                # A's spill stays pending
    assert _ctl(hp, B.HOSTCTL_PENDING_EVENTS) == 1
    a_page = 0
    B.relaygr_kv_alloc(hp.pool, 2, 64, [a_page])                     # B takes A's page ...
    B.relaygr_kv_free(hp.pool, 2)                                    # ... and returns it unused
    B.relaygr_kv_alloc(hp.pool, 4, 64, [1])                          # keep the other page busy
    waits0 = _ctl(hp, B.HOSTCTL_STREAM_WAITS)
    assert B.relaygr_kv_reload_from_host(hp.pool, 3)[0] == B.OK      # C reloads into A's old page
    assert list(B.relaygr_kv_pages(hp.pool, 3)) == [a_page]
    assert _ctl(hp, B.HOSTCTL_STREAM_WAITS) == waits0 + 1            # behind A's pending spill copy
    # relaygr_kv_wait_pages makes the same wait available to a caller that fills pages itself
    _ctl(hp, B.HOSTCTL_COMPLETE_EVENTS, -1)
    B.relaygr_kv_evict(hp.pool, 3, 0)
    B.relaygr_kv_alloc(hp.pool, 5, 64, [a_page])
    waits1 = _ctl(hp, B.HOSTCTL_STREAM_WAITS)
    B.relaygr_kv_wait_pages(hp.pool, 5)
    assert _ctl(hp, B.HOSTCTL_STREAM_WAITS) == waits1                # everything has completed: nothing to wait for
    assert B.relaygr_kv_wait_pages(hp.pool, 77, ok=(B.E_MISS,)) == B.E_MISS


def test_host_pages_stay_behind_a_pending_spill_when_their_user_is_freed():
    hp = HostPool(4, 1)
    _resident(hp, 1, 64, 1)
    _resident(hp, 2, 64, 2)
    _ctl(hp, B.HOSTCTL_MANUAL_EVENTS, 1)
    B.relaygr_kv_evict(hp.pool, 1, 1)                                # spill of user 1 into the only host page: pending
    B.relaygr_kv_free(hp.pool, 1)                                    # the host page is free again, the copy is not done
    waits0 = _ctl(hp, B.HOSTCTL_STREAM_WAITS)
    B.relaygr_kv_evict(hp.pool, 2, 1)                                # user 2 spills into the same host page
    assert _ctl(hp, B.HOSTCTL_STREAM_WAITS) >= waits0 + 1


def test_host_backend_control_is_refused_for_unknown_requests():
    hp = HostPool(2, 0)
    assert B.relaygr_kv_host_backend_control(hp.pool, 99, 0, ok=(B.E_INVALID,))[0] == B.E_INVALID

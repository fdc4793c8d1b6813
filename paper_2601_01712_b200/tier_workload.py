"""The cache-footprint / reload-tier workload (Section 3.4 of the paper: server-local DRAM behind HBM).

A population of users whose aggregate prefix K/V exceeds the HBM budget of the pool is pre-inferred
once and spilled to the pinned-host tier.  Calls of ``batch`` distinct users then arrive with Zipf
popularity.  Before each call the caller does what the paper's pseudo pre-infer step does: probe every
user (HBM, then DRAM), reload DRAM hits on a side stream - evicting least-recently-used residents that
the call does not need when the pool is full (the sliding window) - and then ranks; ``relaygr_rank``
orders itself behind the reload events, so reloads of one call overlap the rank of the previous one.

Only marshalling and policy live here; every byte moved and every score computed is the library's.

    python -m paper_2601_01712_b200.tier_workload --population 1024 --hbm-users 256 --calls 300
"""
from __future__ import annotations

import argparse
import json
from collections import OrderedDict

import numpy as np

from . import binding as B
from . import synth


class ZipfUsers:
    """Users 0..n-1 with popularity proportional to (rank + 1)^-a; draws calls of distinct users."""

    def __init__(self, n: int, a: float):
        p = np.arange(1, n + 1, dtype=np.float64) ** (-a)
        self.p = p / p.sum()
        self.n = n

    def draw_call(self, rng: np.random.Generator, k: int) -> np.ndarray:
        return rng.choice(self.n, size=k, replace=False, p=self.p).astype(np.uint64)


def run(population: int = 1024, hbm_users: int = 256, prefix: int = 4096, batch: int = 32, n_short: int = 64, n_cand: int = 512,
        calls: int = 300, warmup: int = 20, zipf_users: float = 0.9, seed: int = synth.BASE_SEED + 5, shape=None,
        max_in_flight_calls: int = 2, device: str = "cuda:0", collect_scores: bool = False, model=None):
    import time
    import torch
    from . import runtime as rt

    t_setup = time.perf_counter()
    own_model = model is None
    if own_model:
        shape = shape or synth.workload(5).model
        w = synth.make_weights(shape, seed)
        model = rt.Model(shape, w, device)
    else:
        shape, w = model.shape, None
    rng = np.random.default_rng(seed)
    pages_per_user = synth.pages_for(prefix)
    pool = rt.KvPool(model, hbm_users * pages_per_user, population * pages_per_user)
    B.relaygr_kv_set_max_inflight_reloads(pool.pool, max(64, 2 * batch))
    model.reserve(batch * max(prefix, n_short + n_cand), batch, batch * pages_per_user)
    zipf = synth.ZipfIds(shape.vocab, 1.1)
    main, side = torch.cuda.current_stream(), torch.cuda.Stream()
    clock = torch.cuda.Stream()          # carries nothing but the arrival time stamps: an event on an idle stream completes at once

    # ---- every user pre-inferred once, then spilled to the DRAM tier
    for u0 in range(0, population, batch):
        users = np.arange(u0, min(u0 + batch, population), dtype=np.uint64)
        b = synth.make_batch(zipf, rng, [prefix] * len(users), [0] * len(users), [0] * len(users))
        b.users = users
        for u in users:
            pool.alloc(int(u), prefix)
        pool.preinfer(rt.DeviceBatch(b, model.device))
        for u in users:
            pool.evict(int(u), True, side)
    torch.cuda.synchronize()
    st0 = pool.stats()
    setup_s = time.perf_counter() - t_setup

    # ---- the request stream
    lru: "OrderedDict[int, None]" = OrderedDict()          # resident users, least recently used first
    popularity = ZipfUsers(population, zipf_users)
    short_off = np.arange(batch + 1, dtype=np.int32) * n_short
    cand_off = np.arange(batch + 1, dtype=np.int32) * n_cand
    rotations = [(torch.from_numpy(zipf.draw(rng, batch * n_short)).to(model.device),
                  torch.from_numpy(zipf.draw(rng, batch * n_cand)).to(model.device)) for _ in range(8)]
    scores = [torch.empty(batch * n_cand, dtype=torch.float32, device=model.device) for _ in range(max_in_flight_calls + 1)]
    arrive = [torch.cuda.Event(enable_timing=True) for _ in range(warmup + calls)]
    done = [torch.cuda.Event(enable_timing=True) for _ in range(warmup + calls)]
    tiers = {"hbm": 0, "loading": 0, "host": 0}
    kept = []
    t_first = None
    for i in range(warmup + calls):
        if i == warmup:
            torch.cuda.synchronize()
            st_w = pool.stats()
            tiers = {"hbm": 0, "loading": 0, "host": 0}
            t_first = torch.cuda.Event(enable_timing=True)
            t_first.record(main)
        if i >= max_in_flight_calls:
            done[i - max_in_flight_calls].synchronize()         # bounded queue of calls in flight
        users = popularity.draw_call(rng, batch)
        in_call = set(int(u) for u in users)
        # the call's arrival: stamped on the idle stream, so that queueing behind the previous call's reloads counts as latency
        arrive[i].record(clock)
        pages_free = None
        for u in in_call:                                         # the pseudo pre-infer probe: HBM, then DRAM
            tier, _ = pool.lookup(u)
            if tier == B.TIER_HBM:
                tiers["hbm"] += 1
            elif tier == B.TIER_LOADING:
                tiers["loading"] += 1
            elif tier == B.TIER_HOST:
                tiers["host"] += 1
                if pages_free is None:
                    pages_free = pool.stats()["pages_free"]             # read once per call, then counted
                while pages_free < pages_per_user:                       # sliding window: make room
                    victim = next(v for v in lru if v not in in_call)
                    pool.evict(victim, False, side)                       # its DRAM copy stays
                    del lru[victim]
                    pages_free += pages_per_user
                code, _ = pool.reload(u, side)
                assert code == B.OK
                pages_free -= pages_per_user
            else:
                raise RuntimeError("user %d has no cache in any tier" % u)
            lru[u] = None
            lru.move_to_end(u)
        sid, cid = rotations[i % len(rotations)]
        out = scores[i % len(scores)]
        B.relaygr_rank(model.ctx, pool.pool, users, sid.data_ptr(), short_off, cid.data_ptr(), cand_off, out.data_ptr(),
                       main.cuda_stream)
        done[i].record(main)
        if collect_scores:
            kept.append((users.copy(), i % len(rotations), out.clone()))
    t_last = torch.cuda.Event(enable_timing=True)
    t_last.record(main)
    torch.cuda.synchronize()
    assert model.device_status() == 0
    st1 = pool.stats()
    lat = np.array([arrive[i].elapsed_time(done[i]) for i in range(warmup, warmup + calls)])
    wall_ms = t_first.elapsed_time(t_last)
    reload_bytes = st1["reload_bytes"] - st_w["reload_bytes"]
    n_lookups = max(1, sum(tiers.values()))
    report = {
        "workload": "reload tier: %d users x %d-token prefixes (%.1f GiB of K/V in pinned DRAM), HBM pool of %d users (%.1f GiB), "
                    "calls of %d users drawn Zipf(%.1f) without replacement, %d short-term + %d candidates each"
                    % (population, prefix, population * shape.kv_bytes(prefix) / 2**30, hbm_users, hbm_users * shape.kv_bytes(prefix) / 2**30,
                       batch, zipf_users, n_short, n_cand),
        "calls": calls, "rank_latency_ms": {"p50": float(np.percentile(lat, 50)), "p99": float(np.percentile(lat, 99)), "mean": float(lat.mean())},
        "candidates_per_s": calls * batch * n_cand / (wall_ms * 1e-3),
        "hit_rate": {k: v / n_lookups for k, v in tiers.items()},
        "reloads": st1["reloads"] - st_w["reloads"], "reload_bytes": reload_bytes,
        "pcie_gb_per_s": reload_bytes / (wall_ms * 1e-3) / 1e9,
        "hbm_kv_gb_per_s": calls * batch * shape.kv_bytes(prefix) / (wall_ms * 1e-3) / 1e9,
        "spilled_at_start": st0["users_host"], "ms_total": wall_ms, "setup_s": setup_s,
        "latency_clock": "from the call's arrival (an event on an idle stream, before its probes and reloads are enqueued) to the end of its rank",
    }
    result = (report, kept, (model, pool, w, rotations)) if collect_scores else report
    if not collect_scores:
        pool.close()
        if own_model:
            model.close()
    return result


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--population", type=int, default=1024)
    ap.add_argument("--hbm-users", type=int, default=256)
    ap.add_argument("--prefix", type=int, default=4096)
    ap.add_argument("--calls", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=20)
    args = ap.parse_args()
    print(json.dumps(run(population=args.population, hbm_users=args.hbm_users, prefix=args.prefix, calls=args.calls, warmup=args.warmup)))


if __name__ == "__main__":
    main()

"""Two model slots on one GPU: rank on cache for some users while the prefixes of others are pre-inferred.

The paper runs several model slots per special instance so that a long pre-infer does not hold up ranking
(Section 3.2, "Concurrency inside a special instance").  Here a slot is a library context with its own workspace;
both slots share the weights and the prefix-KV pool.  Slot A ranks resident users on a high-priority stream, slot B
pre-infers new users on a low-priority stream into the same pool; the report compares rank latency alone and under
that background load, and gives the pre-infer throughput sustained meanwhile.

    python -m paper_2601_01712_b200.slots_workload --calls 200
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import synth


def run(n_rank_users: int = 32, prefix: int = 2048, n_short: int = 64, n_cand: int = 512, bg_users: int = 8, bg_prefix: int = 8192,
        calls: int = 200, warmup: int = 10, seed: int = synth.BASE_SEED + 6, shape=None, device: str = "cuda:0", return_scores: bool = False):
    import torch
    from . import runtime as rt

    shape = shape or synth.workload(2).model
    rng = np.random.default_rng(seed)
    w = synth.make_weights(shape, seed)
    slot_a = rt.Model(shape, w, device)
    slot_b = slot_a.new_slot()
    zipf = synth.ZipfIds(shape.vocab, 1.1)
    fg = synth.make_batch(zipf, rng, [prefix] * n_rank_users, [n_short] * n_rank_users, [n_cand] * n_rank_users)
    bg = synth.make_batch(zipf, rng, [bg_prefix] * bg_users, [0] * bg_users, [0] * bg_users, first_user=1_000_000)
    pages = n_rank_users * synth.pages_for(prefix) + bg_users * synth.pages_for(bg_prefix)
    pool = rt.KvPool(slot_a, pages)
    slot_a.reserve(n_rank_users * (n_short + n_cand), n_rank_users, n_rank_users * synth.pages_for(prefix))
    slot_a.reserve(n_rank_users * max(prefix, n_short + n_cand), n_rank_users, n_rank_users * synth.pages_for(prefix))
    slot_b.reserve(bg_users * bg_prefix, bg_users, bg_users * synth.pages_for(bg_prefix))
    dfg, dbg = rt.DeviceBatch(fg, slot_a.device), rt.DeviceBatch(bg, slot_a.device)
    lo, hi = torch.cuda.Stream.priority_range()
    s_rank, s_pre = torch.cuda.Stream(priority=hi), torch.cuda.Stream(priority=lo)
    for u in fg.users:
        pool.alloc(int(u), prefix)
    pool.preinfer(dfg, stream=s_rank)
    scores = torch.empty(n_rank_users * n_cand, dtype=torch.float32, device=slot_a.device)

    def timed_rank(n):
        lat = []
        for _ in range(n):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(s_rank)
            pool.rank(dfg, scores, stream=s_rank)
            e1.record(s_rank)
            e1.synchronize()
            lat.append(e0.elapsed_time(e1))
        return np.array(lat)

    timed_rank(warmup)
    alone = timed_rank(calls)
    ref = scores.clone()
    torch.cuda.synchronize()

    # background: slot B keeps pre-inferring the other users' prefixes into the shared pool
    n_pre = 0
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    done = None
    loaded = []
    t0.record(s_pre)
    for i in range(calls):
        if done is None or done.query():                      # one pre-infer call in flight at a time
            if n_pre > 0:
                for u in bg.users:
                    pool.evict(int(u), False, s_pre)
            for u in bg.users:
                pool.alloc(int(u), bg_prefix)
            pool.preinfer(dbg, stream=s_pre, slot=slot_b)
            done = torch.cuda.Event()
            done.record(s_pre)
            n_pre += 1
        loaded.append(timed_rank(1)[0])
    t1.record(s_pre)
    torch.cuda.synchronize()
    same = bool(torch.equal(ref, scores))
    assert slot_a.device_status() == 0 and slot_b.device_status() == 0
    loaded = np.array(loaded)
    span_ms = t0.elapsed_time(t1)
    report = {
        "workload": "slot A ranks %d users x (prefix %d, %d short-term, %d candidates) while slot B pre-infers %d users x %d-token prefixes "
                    "into the same pool" % (n_rank_users, prefix, n_short, n_cand, bg_users, bg_prefix),
        "rank_alone_ms": {"p50": float(np.percentile(alone, 50)), "p99": float(np.percentile(alone, 99))},
        "rank_under_preinfer_ms": {"p50": float(np.percentile(loaded, 50)), "p99": float(np.percentile(loaded, 99))},
        "background_preinfer_calls": n_pre, "background_prefix_tokens_per_s": n_pre * bg_users * bg_prefix / (span_ms * 1e-3),
        "scores_identical_with_and_without_background": same,
    }
    out = (report, ref.cpu().numpy(), fg, w) if return_scores else report
    pool.close(); slot_b.close(); slot_a.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--calls", type=int, default=200)
    ap.add_argument("--bg-users", type=int, default=8)
    ap.add_argument("--bg-prefix", type=int, default=8192)
    args = ap.parse_args()
    print(json.dumps(run(calls=args.calls, bg_users=args.bg_users, bg_prefix=args.bg_prefix)))


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the relay-race GR inference hot path on B200.

One step = one ``relaygr_rank`` call over a batch of the production-shaped workload
(32 users x 2048-token prefix already pre-inferred into the paged pool, 64 short-term
tokens, 512 candidates per user).  The prefix pre-infer and the full recompute of the
same batch are timed beside it.  On one GPU the same line also carries the long-prefix
workload (8 layers, d_model 512; 8192- and 24576-token prefixes), the reload-tier workload
(DRAM tier behind the HBM pool) and single-request latencies.  Prints ONE JSON line.

    python bench.py --gpus 1 --steps 500 --warmup 20
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...   (N independent replicas)
    python bench.py --impl reference      (the CPU checker timed on the host cores)
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "candidates ranked/s with cached prefix KV (rank on cache); p50/p99 rank latency vs full recompute"
UNIT = "candidates/s"
WORKLOAD = "config2: 4 layers, d_model 256, 4 heads x 64, FFN 1024, bf16; 32 users x (prefix 2048 cached, 64 short-term, 512 candidates); Zipf(1.1) ids over 1M items"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the config-2 rank step, from the ncu captures summarised
# under profiles/ (None = no capture of the kernel as it stands).
DRAM_TRAFFIC_BYTES = {"attention": 117.3e6, "gemm": 19.7e6}      # gemm: mean of QKV (9.9 MB) and the fused out-proj + feed-forward kernel (29.6 MB)

MIN_RANK_CALLS, MIN_FULL_CALLS = 500, 100       # individually timed calls behind every p50 / p99 of the main workload


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "tflops_burst": p["bf16_tflops"], "sustained_mhz": (p.get("clocks_under_load") or {}).get("sm_mhz_median"),
                "source": "measured (MEASURED_PEAKS.json)"}
    return {"hbm_gbs": 6650.0, "tflops_sustained": 1400.0, "tflops_burst": 1590.0, "sustained_mhz": 1300.0,
            "source": "fallback (earlier pool measurement)"}


def fractions(tflops, clocks, peaks):
    """A rate against both measured peaks.  The headline fraction takes the peak that was measured at the clock this leg
    ran at: the burst figure when the sampled SM clock stayed near its maximum, the sustained one when the power cap pulled it down."""
    sm, mx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    capped = bool(sm and mx and sm < 0.93 * mx)
    which = "sustained" if capped else "burst"
    return {"tflops": tflops, "frac_burst": tflops / peaks["tflops_burst"], "frac_sustained": tflops / peaks["tflops_sustained"],
            "frac": tflops / peaks["tflops_" + which], "headline_peak": which, "sm_mhz": sm}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def count(self):
        return len(self.rows) if self.proc else 1 << 30

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for name, v in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"], r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def reference_arm(args):
    """The CPU checker as it stands, timed on the host cores on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ref
    from paper_2601_01712_b200 import synth
    wl = synth.workload(2)
    shape = wl.model
    vocab = 50_000       # the sample touches few distinct ids; a smaller table keeps host set-up short
    w = synth.make_weights(shape, wl.seed, vocab=vocab)
    om = ref.Model(shape.n_layers, shape.d_model, shape.n_heads, shape.d_head, shape.d_ff, shape.ln_eps, {**w.mat, **w.vec})
    rng = np.random.default_rng(wl.seed)
    zipf = synth.ZipfIds(vocab, wl.zipf_a)
    P, S, C = 2048, 64, 512
    K, V = om.preinfer(zipf.draw(rng, P))        # not timed: the prefix is cached
    for _ in range(min(args.warmup, 1)):
        om.rank_cached(K, V, zipf.draw(rng, S), zipf.draw(rng, C))
    steps = max(1, min(args.steps, 40))
    t0 = time.perf_counter()
    for _ in range(steps):
        om.rank_cached(K, V, zipf.draw(rng, S), zipf.draw(rng, C))
    dt = (time.perf_counter() - t0) / steps
    val = C / dt
    sample = "1 user per step (prefix 2048 cached by the checker's own pre-infer, 64 short-term, 512 candidates), %d steps" % steps
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": ref.n_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# ---------------------------------------------------------------------------------------------------------------------
# timing helpers (CUDA events on the launching stream)
# ---------------------------------------------------------------------------------------------------------------------
def timed_calls(torch, stream, fn, n, warmup=0):
    """n calls of fn(i), each timed by itself with the stream idle before it (per-call latency as a request sees it).
    Returns (device ms per call, host microseconds spent inside fn per call)."""
    for i in range(warmup):
        fn(i)
    ms, host_us = [], []
    for i in range(n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        t0 = time.perf_counter()
        fn(i)
        host_us.append((time.perf_counter() - t0) * 1e6)
        e1.record(stream)
        e1.synchronize()
        ms.append(e0.elapsed_time(e1))
    return np.array(ms), np.array(host_us)


def pct(a):
    return {"p50": float(np.percentile(a, 50)), "p99": float(np.percentile(a, 99)), "mean": float(np.mean(a)), "n": int(len(a))}


def preinfer_ms(torch, stream, workloads, built, n, warmup=3):
    pool = built.pool
    pool.preinfer(built.dev_batches[0])
    for _ in range(warmup):
        workloads.realloc_users(built)
        pool.preinfer(built.dev_batches[0])
    torch.cuda.synchronize()
    out = []
    for _ in range(n):
        workloads.realloc_users(built)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        pool.preinfer(built.dev_batches[0])
        e1.record(stream)
        e1.synchronize()
        out.append(e0.elapsed_time(e1))
    return np.array(out)


def workload_leg(torch, workloads, shape, peaks, local, model, seed, p_lens, s_lens, c_lens, n_rank, n_full, n_pre, name):
    """Pre-infer, rank on cache and full recompute of one batch, each with its own clock record and roofline fractions."""
    built = workloads.build(shape, seed, p_lens, s_lens, c_lens, n_rotations=4, model=model)
    pool, stream = built.pool, torch.cuda.current_stream()
    b0 = built.batches[0]
    n_cand = int(sum(c_lens))
    scores = torch.empty(max(1, n_cand), dtype=torch.float32, device=model.device)
    nrot = len(built.dev_batches)
    out = {"workload": name, "users": len(p_lens), "prefix_tokens": int(sum(p_lens)), "candidates": n_cand}

    sampler = ClockSampler(local).start()
    pre = preinfer_ms(torch, stream, workloads, built, n_pre)
    clocks = sampler.stop()
    pre_ms = float(np.median(pre))
    out["preinfer"] = {"ms": pre_ms, "tokens_per_s": int(sum(p_lens)) / (pre_ms * 1e-3), "n": int(len(pre)), "clocks": clocks,
                       **fractions(workloads.batch_flops(shape, b0, "preinfer") / (pre_ms * 1e-3) / 1e12, clocks, peaks)}

    sampler = ClockSampler(local).start()
    lat, host = timed_calls(torch, stream, lambda i: pool.rank(built.dev_batches[i % nrot], scores), n_rank, warmup=5)
    clocks = sampler.stop()
    rank_ms = float(np.median(lat))
    out["rank"] = {"ms": rank_ms, "latency_ms": pct(lat), "candidates_per_s": n_cand / (rank_ms * 1e-3), "host_us_per_call": float(np.median(host)),
                   "clocks": clocks, **fractions(workloads.batch_flops(shape, b0, "rank") / (rank_ms * 1e-3) / 1e12, clocks, peaks)}

    sampler = ClockSampler(local).start()
    flat, _ = timed_calls(torch, stream, lambda i: model.rank_full(built.dev_batches[i % nrot], scores), n_full, warmup=2)
    clocks = sampler.stop()
    full_ms = float(np.median(flat))
    out["full_recompute"] = {"ms": full_ms, "latency_ms": pct(flat), "clocks": clocks,
                             **fractions(workloads.batch_flops(shape, b0, "full") / (full_ms * 1e-3) / 1e12, clocks, peaks)}
    out["rank_beats_full_recompute_p99"] = bool(np.percentile(lat, 99) < np.percentile(flat, 99))
    assert model.device_status() == 0, "a kernel reported an internal error"
    built.pool.close()
    del built, scores
    torch.cuda.empty_cache()
    return out


def guarded(fn):
    """A leg that fails must not cost the line: its error is reported in its place."""
    try:
        return fn()
    except Exception as e:      # noqa: BLE001
        return {"error": "%s: %s" % (type(e).__name__, str(e)[:300])}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--lat-calls", type=int, default=0, help="individually timed rank / full-recompute calls behind the percentiles "
                    "(0 = at least 500 / 100; a small number keeps a run under a profiler short)")
    ap.add_argument("--no-legs", action="store_true", help="only the metric's own workload (no long-prefix, reload-tier and single-request legs)")
    ap.add_argument("--tier-population", type=int, default=4096, help="users of the reload-tier leg (their K/V sits in pinned DRAM; 16 MiB each)")
    ap.add_argument("--workload", type=int, default=2, choices=[2, 3, 4],
                    help="2 = production-shaped rank (the metric's workload), 3 = jagged batch with shuffled pages, 4 = long-sequence model")
    ap.add_argument("--users", type=int, default=0, help="0 = the workload's own batch size")
    ap.add_argument("--prefix", type=int, default=0, help="0 = the workload's own prefix length (2048; 8192 for workload 4)")
    ap.add_argument("--candidates", type=int, default=0, help="candidates per user (0 = the workload's own: 512, or 1024 for workload 4)")
    ap.add_argument("--layers", type=int, default=0, help="override the model's depth (sweeps)")
    ap.add_argument("--d-model", type=int, default=0, help="override the model's width (heads of 64, FFN 4x; sweeps)")
    ap.add_argument("--attention", default="softmax", choices=["softmax", "pointwise"],
                    help="pointwise: the HSTU-style SiLU attention variant of the same model (sweeps)")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"], help="f32: the fp32 model and fp32 K/V pages (CUDA-core kernels; sweeps)")
    args = ap.parse_args()
    if args.impl == "reference":
        return reference_arm(args)
    args.warmup = max(args.warmup, 3)

    import torch
    from paper_2601_01712_b200 import build as libbuild
    libbuild.build()
    from paper_2601_01712_b200 import binding as B
    from paper_2601_01712_b200 import replicas, synth, workloads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_mod

    wl = synth.workload(args.workload)
    shape = wl.model
    pointwise = args.attention == "pointwise"
    f32 = args.dtype == "f32"
    if args.layers or args.d_model or pointwise or f32:
        dm = args.d_model or shape.d_model
        shape = synth.ModelShape(args.layers or shape.n_layers, dm, dm // 64, 64, 4 * dm, shape.vocab, synth.DTYPE_F32 if f32 else shape.dtype,
                                 attn_kind=1 if pointwise else 0)
    custom = ("; overrides: layers %d, d_model %d%s%s" % (shape.n_layers, shape.d_model, ", pointwise SiLU attention" if pointwise else "",
                                                          ", fp32 model and fp32 K/V pages" if f32 else "")) \
        if (args.layers or args.d_model or pointwise or f32) else ""
    if args.workload == 3:
        n_users = args.users or 128
        pl, sl, cl = synth.config3_lengths(np.random.default_rng(wl.seed + 1000 * rank), n_users)
        p_lens, s_lens, c_lens = [int(x) for x in pl], [int(x) for x in sl], [int(x) for x in cl]
        workload_name = "config3: config-2 model; %d users, prefix log-uniform [512, 8192] (sum %d), short U[16,128], candidates U[128,1024] (sum %d); pages scattered by a shuffled page table" % (n_users, sum(p_lens), sum(c_lens))
    elif args.workload == 4:
        n_users, P = args.users or 16, args.prefix or 8192
        C = args.candidates or 1024
        p_lens, s_lens, c_lens = [P] * n_users, [128] * n_users, [C] * n_users
        workload_name = "config4: 8 layers, d_model 512, 8 heads x 64, FFN 2048, bf16; %d users x (prefix %d cached, 128 short-term, %d candidates)%s" % (n_users, P, C, custom)
    else:
        n_users, P = args.users or 32, args.prefix or 2048
        C = args.candidates or 512
        p_lens, s_lens, c_lens = [P] * n_users, [64] * n_users, [C] * n_users
        workload_name = WORKLOAD if (n_users, P, C, custom) == (32, 2048, 512, "") else \
            "config2 model; %d users x (prefix %d cached, 64 short-term, %d candidates)%s" % (n_users, P, C, custom)
    # replicas: every rank holds the users that hash to it (affinity routing by user id), no data-path collective
    user_ids, u = [], 0
    while len(user_ids) < n_users:
        if replicas.owner_rank(u, world) == rank:
            user_ids.append(u)
        u += 1
    built = workloads.build(shape, wl.seed + 1000 * rank, p_lens, s_lens, c_lens, n_rotations=8, shuffle_pages=args.workload == 3,
                            user_ids=user_ids, device="cuda:%d" % local)
    model, pool = built.model, built.pool
    stream = torch.cuda.current_stream()
    n_cand = int(sum(c_lens))
    scores = torch.empty(n_cand, dtype=torch.float32, device=model.device)
    peaks = load_peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return replicas.max_over_ranks(ms, dist, model.device)

    # ---- pre-infer (timed beside the metric) --------------------------------------------------------
    pre_steps = max(3, min(20, args.steps // 20))        # 20 timed calls at the default --steps
    sampler = ClockSampler(local).start()
    pre_ms = preinfer_ms(torch, stream, workloads, built, pre_steps)
    pre_clocks = sampler.stop()
    pre_ms_med = float(np.median(pre_ms))
    # per-kernel-class timing of pre-infer (events around every launch; separate from the timing above)
    B.relaygr_profile_enable(model.ctx, True)
    for _ in range(2):
        workloads.realloc_users(built)
        pool.preinfer(built.dev_batches[0])
    pre_prof = B.relaygr_profile_read(model.ctx)
    B.relaygr_profile_enable(model.ctx, False)
    pre_kernel_ms = {k: pre_prof[k] / 2 for k in pre_prof if k.endswith("_ms")}

    # ---- rank on cache: the metric ------------------------------------------------------------------
    nrot = len(built.dev_batches)
    for i in range(args.warmup):
        pool.rank(built.dev_batches[i % nrot], scores)
    launches0 = model.launch_count()
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    evs[0].record(stream)
    for i in range(args.steps):
        pool.rank(built.dev_batches[i % nrot], scores)
        evs[i + 1].record(stream)
    barrier()
    torch.cuda.synchronize()
    launches = model.launch_count() - launches0
    # a timed region shorter than a few sampling periods: keep the same load running (untimed) until the sampler has seen it
    extra = 0
    while sampler.count() < 3 and extra < 20000:
        pool.rank(built.dev_batches[extra % nrot], scores)
        extra += 1
        if extra % 50 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    total_ms = max_over_ranks(evs[0].elapsed_time(evs[-1]))
    lat = np.array([evs[i].elapsed_time(evs[i + 1]) for i in range(args.steps)])
    assert model.device_status() == 0, "a kernel reported an internal error"
    ms_per_step = total_ms / args.steps
    value = world * n_cand / (ms_per_step * 1e-3)

    # one call at a time (stream idle before each call): per-call latency as a request sees it, and the host's share of it
    n_lat = args.lat_calls or (max(MIN_RANK_CALLS, min(args.steps, 2000)) if ms_per_step < 20 else max(100, min(args.steps, 500)))
    lat1, host_us = timed_calls(torch, stream, lambda i: pool.rank(built.dev_batches[i % nrot], scores), n_lat)

    # ---- full recompute of the same batches ---------------------------------------------------------
    n_full = args.lat_calls or (MIN_FULL_CALLS if ms_per_step < 20 else 20)
    full_lat, _ = timed_calls(torch, stream, lambda i: model.rank_full(built.dev_batches[i % nrot], scores), n_full, warmup=3)

    # ---- per-kernel timing of the rank step (events around every launch; separate from the timed region)
    B.relaygr_profile_enable(model.ctx, True)
    prof_steps = min(args.steps, 50)
    for i in range(prof_steps):
        pool.rank(built.dev_batches[i % nrot], scores)
    prof = B.relaygr_profile_read(model.ctx)
    B.relaygr_profile_enable(model.ctx, False)
    prof_total = sum(prof[k] for k in prof if k.endswith("_ms"))
    b0 = built.batches[0]
    # algorithmic FLOPs of the two tensor-core kernel classes over one rank step (dead last-layer work excluded)
    attn_flops_step = workloads.batch_flops(shape, b0, "rank") - workloads.batch_linear_flops(shape, b0, "rank")
    class_flops = {"attention": attn_flops_step, "gemm": workloads.batch_linear_flops(shape, b0, "rank")}
    class_name = {"attention": "attention_tc_kernel (rank on cache)", "gemm": "gemm_tc_kernel + ffn_fused_kernel (QKV; out-proj + feed-forward of the rank step)"}
    rooflines = {}
    for cls in ("attention", "gemm"):
        n_launch = max(1, prof[cls + "_launches"])
        ms = prof[cls + "_ms"] / n_launch                       # average launch duration, CUDA events on the launching stream
        fl = class_flops[cls] * prof_steps / n_launch           # algorithmic FLOPs per launch
        tf = fl / (ms * 1e-3) / 1e12
        fr = fractions(tf, clocks, peaks)
        rooflines[cls] = {"kernel": class_name[cls], "bound": "tensor", "achieved": tf, "peak": peaks["tflops_" + fr["headline_peak"]], "unit": "TFLOP/s",
                          "frac": fr["frac"], "frac_burst": fr["frac_burst"], "frac_sustained": fr["frac_sustained"],
                          "peak_source": "%s, %s bf16 figure (median SM clock of the timed region %s MHz)" % (peaks["source"], fr["headline_peak"], fr["sm_mhz"]),
                          "traffic": DRAM_TRAFFIC_BYTES[cls] if workload_name == WORKLOAD else None,
                          "ms_per_launch": ms, "launches_per_step": n_launch / prof_steps, "algorithmic_flops_per_launch": fl,
                          "share_of_step": prof[cls + "_ms"] / prof_total if prof_total else None}
    dominant = max(rooflines, key=lambda c: rooflines[c]["share_of_step"] or 0.0)
    other = "gemm" if dominant == "attention" else "attention"

    # ---- end to end through host buffers ------------------------------------------------------------
    hb = [(torch.from_numpy(b.short_ids).pin_memory(), torch.from_numpy(b.cand_ids).pin_memory()) for b in built.batches]
    # Two calls are kept in flight, as a serving loop would: while call i runs on the GPU the host launches call i + 1 and
    # then reads the result of call i - 1 (every call's inputs are copied from pinned host memory and every call's result
    # is copied back and looked at by the host, all inside the timed region; buffers alternate).  The strictly serial form -
    # the host waits for each result before it launches the next call - is timed too ("ms_per_step_serial").
    d_short = [torch.empty_like(built.dev_batches[0].short_ids) for _ in range(2)]
    d_cand = [torch.empty_like(built.dev_batches[0].cand_ids) for _ in range(2)]
    d_scores = [torch.empty_like(scores) for _ in range(2)]
    h_scores = [torch.empty(n_cand, dtype=torch.float32).pin_memory() for _ in range(2)]
    done = [torch.cuda.Event() for _ in range(2)]
    ctx, kp = model.ctx, pool.pool
    seen = [0.0]

    def e2e_launch(i):
        k = i & 1
        hs, hc = hb[i % nrot]
        d_short[k].copy_(hs, non_blocking=True)
        d_cand[k].copy_(hc, non_blocking=True)
        B.relaygr_rank(ctx, kp, b0.users, d_short[k].data_ptr(), b0.short_off, d_cand[k].data_ptr(), b0.cand_off,
                       d_scores[k].data_ptr(), stream.cuda_stream)
        h_scores[k].copy_(d_scores[k], non_blocking=True)
        done[k].record(stream)

    def e2e_read(i):
        k = i & 1
        done[k].synchronize()
        seen[0] += float(h_scores[k][0])             # the host looks at the result

    def e2e_run(n, depth):
        for i in range(n):
            e2e_launch(i)
            if depth == 1:
                e2e_read(i)
            elif i > 0:
                e2e_read(i - 1)
        if depth > 1:
            e2e_read(n - 1)

    e2e_steps = min(args.steps, 200)
    e2e_times = {}
    for depth in (1, 2):
        e2e_run(5, depth)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        e2e_run(e2e_steps, depth)                    # (returns after the host has read the last result)
        e1.record(stream)
        barrier()
        e2e_times[depth] = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps
    e2e_ms = e2e_times[2]
    e2e = {"value": world * n_cand / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms, "calls_in_flight": 2,
           "ms_per_step_serial": e2e_times[1], "value_serial": world * n_cand / (e2e_times[1] * 1e-3),
           "h2d_bytes_per_step": int(hb[0][0].numel() * 4 + hb[0][1].numel() * 4), "d2h_bytes_per_step": int(n_cand * 4)}

    # ---- CPU baseline: the checker, timed on this machine's host cores ----------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.workload == 2 and not f32:
        from oracle import ref
        om = ref.Model(shape.n_layers, shape.d_model, shape.n_heads, shape.d_head, shape.d_ff, shape.ln_eps,
                       {**built.weights.mat, **built.weights.vec})
        n_sample = 10                                               # ~11 s of timed CPU work on 16 cores
        t_cpu, err, n_scored = 0.0, 0.0, 0
        for u in range(n_sample):
            p, _, _ = b0.user_slices(u)
            K, V = om.preinfer(p)                                   # untimed: the prefix is cached
            for r in range(nrot):                                   # the same user with every rotation of short-term / candidate ids
                br = built.batches[r]
                _, s_ids, c_ids = br.user_slices(u)
                t0 = time.perf_counter()
                want = om.rank_cached(K, V, s_ids, c_ids)
                t_cpu += time.perf_counter() - t0
                n_scored += len(c_ids)
                if r < 2:
                    pool.rank(built.dev_batches[r], scores)
                    got = scores.cpu().numpy()
                    err = max(err, float(np.max(np.abs(got[br.cand_off[u]:br.cand_off[u + 1]] - want))))
        cpu = {"value": n_scored / t_cpu, "unit": UNIT, "cores": ref.n_threads(), "kind": "oracle",
               "sample": "%d of the %d users of the batch x %d rotations of their short-term / candidate ids, rank on cache only "
                         "(prefix K/V from the checker's own pre-infer, untimed); %.1f s of CPU work" % (n_sample, n_users, nrot, t_cpu),
               "max_abs_err_vs_gpu": err}

    rank_flops = workloads.batch_flops(shape, b0, "rank")
    pre_flops = workloads.batch_flops(shape, b0, "preinfer")
    full_flops = workloads.batch_flops(shape, b0, "full")
    full_med = float(np.median(full_lat))

    # ---- further legs (one GPU, the metric's own workload only): single requests, long prefixes, the reload tier --------
    legs = {}
    if world == 1 and not args.no_legs and args.workload == 2 and not custom and (args.users, args.prefix, args.candidates) == (0, 0, 0):
        def b1(model_, shape_, seed, P_, S_, C_, name):
            return workload_leg(torch, workloads, shape_, peaks, local, model_, seed, [P_], [S_], [C_], MIN_RANK_CALLS, MIN_FULL_CALLS, 20, name)

        legs["b1"] = {"config2": guarded(lambda: b1(model, shape, wl.seed + 7, 2048, 64, 512,
                                                     "one request: config-2 model, one user (prefix 2048 cached, 64 short-term, 512 candidates)"))}
        # the reload tier on the same model (its users' prefixes are 4096 tokens: 16 MiB of K/V each)
        def tier():
            from paper_2601_01712_b200 import tier_workload
            last = None
            for pop in (args.tier_population, args.tier_population // 2, args.tier_population // 4):      # the largest population the box can pin
                try:
                    rep = tier_workload.run(population=pop, hbm_users=pop // 4, calls=300, warmup=20, model=model)
                    rep["population_tried_first"] = args.tier_population
                    return rep
                except RuntimeError as e:       # pinned allocation refused: halve
                    last = e
                    torch.cuda.empty_cache()
            raise last
        built.pool.close()
        del built, pool
        torch.cuda.empty_cache()
        sampler = ClockSampler(local).start()
        legs["tier"] = guarded(tier)
        if isinstance(legs["tier"], dict):
            legs["tier"]["clocks"] = sampler.stop()
        model.close()
        del model
        torch.cuda.empty_cache()

        def long_prefix():
            from paper_2601_01712_b200 import runtime as rt
            wl4 = synth.workload(4)
            w4 = synth.make_weights(wl4.model, wl4.seed)
            m4 = rt.Model(wl4.model, w4, "cuda:%d" % local)
            del w4
            out = {}
            for P_, n_rank, n_full, n_pre in ((8192, 200, 20, 20), (24576, 100, 10, 20)):
                out["P%d" % P_] = guarded(lambda: workload_leg(
                    torch, workloads, wl4.model, peaks, local, m4, wl4.seed + P_, [P_] * 16, [128] * 16, [1024] * 16, n_rank, n_full, n_pre,
                    "config4: 8 layers, d_model 512, 8 heads x 64, FFN 2048, bf16; 16 users x (prefix %d cached, 128 short-term, 1024 candidates)" % P_))
            legs["b1"]["config4"] = guarded(lambda: workload_leg(
                torch, workloads, wl4.model, peaks, local, m4, wl4.seed + 9, [8192], [128], [1024], MIN_RANK_CALLS, MIN_FULL_CALLS, 20,
                "one request: config-4 model, one user (prefix 8192 cached, 128 short-term, 1024 candidates)"))
            m4.close()
            return out
        legs["long_prefix"] = guarded(long_prefix)

    if rank == 0:
        rank_fr = fractions(rank_flops / (ms_per_step * 1e-3) / 1e12, clocks, peaks)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if f32 else "bf16", "data": "synthetic",
            "config": {"workload": workload_name, "step": "one relaygr_rank call over the batch, prefix KV already in the paged pool",
                       "users": n_users, "prefix_tokens": int(sum(p_lens)), "short_tokens": int(sum(s_lens)), "candidates": n_cand,
                       "l2": "inputs larger than L2: each step streams %.0f MiB of prefix K/V and rotates 8 input sets" % (shape.kv_bytes(int(sum(p_lens))) / 2**20),
                       "parallelism": "replicas (users placed by replicas.owner_rank(user id)), no collective" if world > 1 else "single GPU"},
            "latency_ms": {"rank_p50_backlogged": float(np.percentile(lat, 50)), "rank_p99_backlogged": float(np.percentile(lat, 99)),
                           "rank_p50": float(np.percentile(lat1, 50)), "rank_p99": float(np.percentile(lat1, 99)), "rank_calls": int(len(lat1)),
                           "full_recompute_p50": float(np.percentile(full_lat, 50)), "full_recompute_p99": float(np.percentile(full_lat, 99)),
                           "full_recompute_calls": int(len(full_lat)),
                           "rank_beats_full_recompute_p99": bool(np.percentile(lat1, 99) < np.percentile(full_lat, 99))},
            "host_us_per_rank_call": float(np.median(host_us)),
            "preinfer": {"tokens_per_s": int(sum(p_lens)) / (pre_ms_med * 1e-3), "ms": pre_ms_med, "calls": int(len(pre_ms)), "clocks": pre_clocks,
                         **fractions(pre_flops / (pre_ms_med * 1e-3) / 1e12, pre_clocks, peaks),
                         "kernel_ms": pre_kernel_ms},
            "whole_step_roofline": {"rank": rank_fr,
                                    "full_recompute": fractions(full_flops / (full_med * 1e-3) / 1e12, clocks, peaks)},
            "roofline": rooflines[dominant], "roofline_second_kernel": rooflines[other],
            "kernel_ms_per_step": {k: prof[k] / prof_steps for k in prof if k.endswith("_ms")},
            "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "cpu_baseline": cpu,
        }
        out.update(legs)
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

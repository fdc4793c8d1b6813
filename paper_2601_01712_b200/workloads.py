"""The evaluation workloads as device objects, and the algorithmic work they contain.

Argument marshalling and bookkeeping only: models, pools and batches are built from
``synth`` and handed to the C-ABI library through ``runtime``.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np

from . import synth


# ---------------------------------------------------------------------------------------------
# Algorithmic FLOPs (what the method must do; dead last-layer work excluded).  Per token-layer
# the linear maps cost 6d^2 (QKV) + 2d^2 (out) + 4dF (FFN); attention costs 4*d per visible
# (query, key) pair (QK^T and PV, all heads).
# ---------------------------------------------------------------------------------------------
def linear_flops_per_token(shape: synth.ModelShape) -> float:
    d, F = shape.d_model, shape.d_ff
    return 8.0 * d * d + 4.0 * d * F


def pairs_preinfer(P: int) -> float:
    return P * (P + 1) / 2.0


def pairs_rank(P: int, S: int, C: int) -> float:
    return S * P + S * (S + 1) / 2.0 + C * (P + S + 1)


def pairs_full(P: int, S: int, C: int) -> float:
    return (P + S) * (P + S + 1) / 2.0 + C * (P + S + 1)


def flops_preinfer(shape: synth.ModelShape, P: int) -> float:
    L, d = shape.n_layers, shape.d_model
    return (L - 1) * (linear_flops_per_token(shape) * P + 4.0 * d * pairs_preinfer(P)) + 4.0 * d * d * P


def flops_rank(shape: synth.ModelShape, P: int, S: int, C: int) -> float:
    L, d = shape.n_layers, shape.d_model
    lin = linear_flops_per_token(shape)
    last = 4.0 * d * d * S + lin * C + 4.0 * d * C * (P + S + 1)
    return (L - 1) * (lin * (S + C) + 4.0 * d * pairs_rank(P, S, C)) + last


def flops_full(shape: synth.ModelShape, P: int, S: int, C: int) -> float:
    L, d = shape.n_layers, shape.d_model
    lin = linear_flops_per_token(shape)
    last = 4.0 * d * d * (P + S) + lin * C + 4.0 * d * C * (P + S + 1)
    return (L - 1) * (lin * (P + S + C) + 4.0 * d * pairs_full(P, S, C)) + last


def attention_flops_per_layer(shape: synth.ModelShape, batch: synth.Batch, mode: str) -> float:
    """Algorithmic attention FLOPs of ONE layer's attention launch over the whole batch."""
    tot = 0.0
    for i in range(batch.n_users):
        P = int(batch.prefix_off[i + 1] - batch.prefix_off[i])
        S = int(batch.short_off[i + 1] - batch.short_off[i])
        C = int(batch.cand_off[i + 1] - batch.cand_off[i])
        pairs = {"preinfer": pairs_preinfer(P), "rank": pairs_rank(P, S, C), "full": pairs_full(P, S, C)}[mode]
        tot += 4.0 * shape.d_model * pairs
    return tot


def batch_linear_flops(shape: synth.ModelShape, batch: synth.Batch, mode: str) -> float:
    """Algorithmic FLOPs of the linear maps (QKV, out-proj, FFN) of one call: ``batch_flops`` minus attention."""
    L, d = shape.n_layers, shape.d_model
    lin = linear_flops_per_token(shape)
    tot = 0.0
    for i in range(batch.n_users):
        P = int(batch.prefix_off[i + 1] - batch.prefix_off[i])
        S = int(batch.short_off[i + 1] - batch.short_off[i])
        C = int(batch.cand_off[i + 1] - batch.cand_off[i])
        if mode == "preinfer":
            tot += (L - 1) * lin * P + 4.0 * d * d * P
        elif mode == "rank":
            tot += (L - 1) * lin * (S + C) + 4.0 * d * d * S + lin * C
        else:
            tot += (L - 1) * lin * (P + S + C) + 4.0 * d * d * (P + S) + lin * C
    return tot


def batch_flops(shape: synth.ModelShape, batch: synth.Batch, mode: str) -> float:
    tot = 0.0
    for i in range(batch.n_users):
        P = int(batch.prefix_off[i + 1] - batch.prefix_off[i])
        S = int(batch.short_off[i + 1] - batch.short_off[i])
        C = int(batch.cand_off[i + 1] - batch.cand_off[i])
        tot += {"preinfer": flops_preinfer(shape, P), "rank": flops_rank(shape, P, S, C),
                "full": flops_full(shape, P, S, C)}[mode]
    return tot


# ---------------------------------------------------------------------------------------------
@dataclass
class Built:
    shape: synth.ModelShape
    weights: synth.Weights
    model: object            # runtime.Model
    pool: object             # runtime.KvPool
    batches: List[synth.Batch]          # same users / prefixes, rotating short-term + candidate ids
    dev_batches: List[object]           # runtime.DeviceBatch


def build(shape: synth.ModelShape, seed: int, p_lens, s_lens, c_lens, n_rotations: int = 8, zipf_a: float = 1.1,
          shuffle_pages: bool = False, spare_pages: int = 0, host_pages: int = 0, first_user: int = 0,
          weights: Optional[synth.Weights] = None, device: str = "cuda:0", model=None, user_ids=None) -> Built:
    """Model + pool + ``n_rotations`` batches with the given per-user lengths; users are ALLOCATED
    (not yet pre-inferred).  ``shuffle_pages`` scatters each user's pages with a seeded shuffle.
    ``model``: reuse an existing runtime.Model (its weights and context) instead of uploading a new one.
    ``user_ids``: the users' ids (default: first_user, first_user + 1, ...)."""
    from . import runtime as rt
    if model is not None:
        w = weights
    else:
        w = weights if weights is not None else synth.make_weights(shape, seed)
        model = rt.Model(shape, w, device)
    rng = np.random.default_rng(seed)
    zipf = synth.ZipfIds(shape.vocab, zipf_a)
    first = synth.make_batch(zipf, rng, p_lens, s_lens, c_lens, first_user)
    if user_ids is not None:
        assert len(user_ids) == len(p_lens) and len(set(int(u) for u in user_ids)) == len(p_lens)
        first.users = np.asarray(user_ids, dtype=np.uint64)
    batches = [first] + [synth.draw_short_cand(zipf, rng, first) for _ in range(n_rotations - 1)]
    counts = [synth.pages_for(p) for p in p_lens]
    total = sum(counts) + spare_pages
    pool = rt.KvPool(model, total, host_pages)
    ids = synth.shuffled_pages(np.random.default_rng(seed + 1), total, counts) if shuffle_pages else [None] * len(counts)
    for i, u in enumerate(first.users):
        pool.alloc(u, p_lens[i], ids[i])
    rows = int(sum(p_lens) + sum(s_lens) + sum(c_lens))
    model.reserve(rows, len(p_lens), sum(counts))
    dev = [rt.DeviceBatch(b, model.device) for b in batches]
    return Built(shape, w, model, pool, batches, dev)


def realloc_users(built: Built):
    """Put every user back to ALLOCATED on the same pages (for repeated pre-infer timing)."""
    b = built.batches[0]
    pages = [built.pool.pages(u) for u in b.users]
    for u in b.users:
        built.pool.evict(u, False)
    for i, u in enumerate(b.users):
        built.pool.alloc(u, int(b.prefix_off[i + 1] - b.prefix_off[i]), pages[i])

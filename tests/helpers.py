"""Shared helpers for the GPU parity tests: build the CPU checker and the CUDA model from
the same synthetic weights, and run both on the same jagged batch."""
import numpy as np

from oracle import ref
from paper_2601_01712_b200 import synth
from tests import bf16_noise

TOL_F32 = 1e-4      # fp32 model: max-abs score error against the fp64 checker
TOL_BF16 = 2e-2     # bf16 model: same, the checker reading the bf16-rounded parameters (the bound of the named workloads)


def oracle_model(shape: synth.ModelShape, w: synth.Weights) -> ref.Model:
    return ref.Model(shape.n_layers, shape.d_model, shape.n_heads, shape.d_head, shape.d_ff, shape.ln_eps,
                     {**w.mat, **w.vec}, attn_kind=shape.attn_kind)


def oracle_scores(om: ref.Model, batch: synth.Batch, users=None, cached: bool = True):
    """Scores per user (list of arrays) from the checker; ``users`` selects a subset."""
    out = {}
    for i in (range(batch.n_users) if users is None else users):
        p, s, c = batch.user_slices(i)
        if cached:
            K, V = om.preinfer(p)
            out[i] = om.rank_cached(K, V, s, c)
        else:
            out[i] = om.full(p, s, c)
    return out


def max_abs_err(gpu_scores: np.ndarray, batch: synth.Batch, want: dict) -> float:
    worst = 0.0
    for i, w in want.items():
        g = gpu_scores[batch.cand_off[i]:batch.cand_off[i + 1]]
        assert g.shape == w.shape
        if len(w):
            assert np.all(np.isfinite(g)), "non-finite GPU score"
            worst = max(worst, float(np.max(np.abs(g.astype(np.float64) - w))))
    return worst


def small_bf16_shape(vocab=5000, layers=2, d=256, heads=4, ff=512, attn_kind=0):
    return synth.ModelShape(layers, d, heads, d // heads, ff, vocab, synth.DTYPE_BF16, attn_kind=attn_kind)


def bf16_noise_bounds(shape: synth.ModelShape, w: synth.Weights, batch: synth.Batch, want: dict):
    """Bounds for shapes other than the named workloads, derived from the arithmetic rather than from a run of the kernels.

    A bf16 tensor-core model must round six kinds of values per layer (the operands of its matrix products: LayerNorm
    outputs, q / k / v, the attention weights, the attention output, the hidden activations; ``tests/bf16_noise.py``).  Each
    adds a comparable share of noise to the scores (0.001-0.003 rms on scores of unit scale), none dominates, and none can be
    left out.  The emulation there rounds at exactly these sites and nowhere else; its error against the checker is a sample of
    that noise for THIS model and batch.  With sigma its root mean square:
      * the largest of a few hundred to a thousand errors of such noise sits at 3-4 sigma, so the maximum is bounded by
        5 sigma - or by the named workloads' 2e-2 where that is larger;
      * the kernels' own rms error may exceed sigma by the small approximations they add (ex2.approx, tanh.approx, the cubic
        exponential: each below the bf16 rounding it feeds): bounded by 1.5 sigma.
    Returns (bound on the maximum, bound on the rms, sigma)."""
    sd = dict(n_layers=shape.n_layers, d_model=shape.d_model, n_heads=shape.n_heads, d_head=shape.d_head, ln_eps=shape.ln_eps,
              attn_kind=shape.attn_kind)
    params = {**w.mat, **w.vec}
    err = []
    for i, wv in want.items():
        p, s, c = batch.user_slices(i)
        if len(c):
            err.append(bf16_noise.scores(sd, params, p, s, c) - wv)
    sigma = float(np.sqrt(np.mean(np.concatenate(err) ** 2))) if err else 0.0
    return max(TOL_BF16, 5.0 * sigma), 1.5 * sigma + 2e-4, sigma

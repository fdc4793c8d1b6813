"""Shared helpers for the GPU parity tests: build the CPU checker and the CUDA model from
the same synthetic weights, and run both on the same jagged batch."""
import numpy as np

from oracle import ref
from paper_2601_01712_b200 import synth

TOL_F32 = 1e-4      # fp32 model: max-abs score error against the fp64 checker
TOL_BF16 = 2e-2     # bf16 model: same, the checker reading the bf16-rounded parameters
# The pointwise-attention variant of the same synthetic weights spreads its scores twice as wide (std ~0.7 against ~0.35:
# no softmax bounds the attention output), and the bf16 roundings of operands and of P are relative errors, so its
# absolute score error doubles too (measured rms 0.005 against 0.003).  Same relative accuracy, twice the absolute bound.
TOL_BF16_POINTWISE = 4e-2


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

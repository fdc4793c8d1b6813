"""Pins for the CPU checker's pointwise (HSTU-style) attention, CPU only.

The variant replaces the softmax over a query's allowed keys by an elementwise
SiLU and divides by the number of allowed keys (the checker's header states the
readings).  It is pinned the same way as the softmax path: a dense-mask brute
force written separately, the defining relation rank-on-cache == full
inference, a closed form that fixes both the SiLU and the normaliser, and
planted mistakes that each of those must catch.
"""
import numpy as np
import pytest

from oracle import ref
from paper_2601_01712_b200 import synth
from tests import brute_force

pytestmark = pytest.mark.filterwarnings("ignore")


def tiny_shape(L=2, d=16, H=2, F=32, vocab=50):
    return synth.ModelShape(L, d, H, d // H, F, vocab, synth.DTYPE_F32, attn_kind=1)


def make_model(shape, seed, override=None, attn_kind=1):
    w = synth.make_weights(shape, seed)
    params = {**w.mat, **w.vec}
    if override:
        params.update(override)
    return ref.Model(shape.n_layers, shape.d_model, shape.n_heads, shape.d_head, shape.d_ff, shape.ln_eps, params,
                     attn_kind=attn_kind), params


def shape_dict(shape, attn_kind=1):
    return dict(n_layers=shape.n_layers, d_model=shape.d_model, n_heads=shape.n_heads, d_head=shape.d_head,
                ln_eps=shape.ln_eps, attn_kind=attn_kind)


def ids(rng, n, vocab=50):
    return rng.integers(0, vocab, n).astype(np.int32)


@pytest.mark.parametrize("P,S,C", [(16, 4, 4), (9, 0, 3), (5, 3, 1), (1, 0, 1), (7, 1, 5)])
def test_full_matches_dense_mask_brute_force(P, S, C):
    shape = tiny_shape()
    m, params = make_model(shape, 3)
    rng = np.random.default_rng(500 + P + S + C)
    p, s, c = ids(rng, P), ids(rng, S), ids(rng, C)
    got = m.full(p, s, c)
    want = brute_force.scores(shape_dict(shape), params, p, s, c)
    assert np.max(np.abs(got - want)) <= 1e-10
    # and it is not the softmax model
    soft, _ = make_model(shape, 3, attn_kind=0)
    assert np.max(np.abs(soft.full(p, s, c) - got)) > 1e-3


@pytest.mark.parametrize("P,S,C", [(16, 4, 4), (40, 0, 6), (33, 7, 1), (1, 2, 3)])
def test_rank_on_cached_prefix_equals_full_inference(P, S, C):
    shape = tiny_shape(L=3)
    m, _ = make_model(shape, 6)
    rng = np.random.default_rng(P * 37 + S)
    p, s, c = ids(rng, P), ids(rng, S), ids(rng, C)
    K, V = m.preinfer(p)
    assert np.max(np.abs(m.rank_cached(K, V, s, c) - m.full(p, s, c))) <= 1e-10


def test_candidates_do_not_see_one_another():
    shape = tiny_shape()
    m, _ = make_model(shape, 8)
    rng = np.random.default_rng(5)
    p, s, c = ids(rng, 12), ids(rng, 3), ids(rng, 6)
    base = m.full(p, s, c)
    c2 = c.copy()
    c2[1:] = (c2[1:] + 7) % 50
    assert abs(m.full(p, s, c2)[0] - base[0]) <= 1e-12


def _closed_form_scores(shape, params, p, s, c, weight_of_pair, count_of):
    """One layer whose every logit is the same constant z: o_t = weight_of_pair(z) * sum of allowed v / count_of(n_allowed)."""
    d, dh = shape.d_model, shape.d_head
    f64 = lambda a: np.asarray(a, dtype=np.float64)
    ln = lambda z, g, b: (z - z.mean(-1, keepdims=True)) / np.sqrt(z.var(-1, keepdims=True) + shape.ln_eps) * g + b
    ids_all = np.concatenate([p, s, c])
    x = f64(params["emb"])[ids_all]
    a = ln(x, f64(params["ln1_g"][0]), f64(params["ln1_b"][0]))
    v = a @ f64(params["w_qkv"][0][2 * d:]).T + f64(params["b_qkv"][0][2 * d:])
    bq, bk = f64(params["b_qkv"][0][:d]), f64(params["b_qkv"][0][d:2 * d])
    out = []
    for i in range(len(c)):
        t = len(p) + len(s) + i
        n_allowed = len(p) + len(s) + 1
        o = np.zeros(d)
        for h in range(shape.n_heads):
            sl = slice(h * dh, (h + 1) * dh)
            z = float(bq[sl] @ bk[sl]) / np.sqrt(dh)
            o[sl] = weight_of_pair(z) * (v[:len(p) + len(s), sl].sum(0) + v[t, sl]) / count_of(n_allowed)
        hmid = x[t] + o @ f64(params["w_o"][0]).T + f64(params["b_o"][0])
        zz = ln(hmid, f64(params["ln2_g"][0]), f64(params["ln2_b"][0])) @ f64(params["w1"][0]).T + f64(params["b1"][0])
        xx = hmid + (zz / (1 + np.exp(-zz))) @ f64(params["w2"][0]).T + f64(params["b2"][0])
        out.append(ln(xx, f64(params["lnf_g"]), f64(params["lnf_b"])) @ f64(params["w_score"]) + params["b_score"][0])
    return np.array(out)


def _constant_logit_model(seed=12):
    """W_q = W_k = 0 with non-zero query / key biases: q.k is the same for every pair of a head."""
    shape = tiny_shape(L=1)
    w = synth.make_weights(shape, seed)
    d = shape.d_model
    wq = w.mat["w_qkv"].copy()
    wq[:, :2 * d, :] = 0.0
    bq = w.vec["b_qkv"].copy()
    rng = np.random.default_rng(99)
    bq[:, :2 * d] = rng.normal(0.0, 1.0, (1, 2 * d)).astype(np.float32)
    return shape, {"w_qkv": wq, "b_qkv": bq}


def test_constant_logits_give_silu_times_mean_of_values():
    shape, ov = _constant_logit_model()
    m, params = make_model(shape, 12, ov)
    rng = np.random.default_rng(24)
    p, s, c = ids(rng, 8), ids(rng, 2), ids(rng, 3)
    want = _closed_form_scores(shape, params, p, s, c, lambda z: z / (1.0 + np.exp(-z)), lambda n: n)
    assert np.max(np.abs(m.full(p, s, c) - want)) <= 1e-10


@pytest.mark.parametrize("mistake", ["sigmoid_only", "count_all_tokens", "no_scale", "no_normaliser"])
def test_closed_form_catches_planted_mistakes(mistake):
    """Each plausible slip in the pointwise aggregation moves the closed form away from the checker."""
    shape, ov = _constant_logit_model()
    m, params = make_model(shape, 12, ov)
    rng = np.random.default_rng(24)
    p, s, c = ids(rng, 8), ids(rng, 2), ids(rng, 3)
    T = len(p) + len(s) + len(c)
    sq = np.sqrt(shape.d_head)
    wrong = {
        "sigmoid_only": (lambda z: 1.0 / (1.0 + np.exp(-z)), lambda n: n),
        "count_all_tokens": (lambda z: z / (1.0 + np.exp(-z)), lambda n: T),
        "no_scale": (lambda z: (z * sq) / (1.0 + np.exp(-z * sq)), lambda n: n),
        "no_normaliser": (lambda z: z / (1.0 + np.exp(-z)), lambda n: 1),
    }[mistake]
    bad = _closed_form_scores(shape, params, p, s, c, *wrong)
    assert np.max(np.abs(m.full(p, s, c) - bad)) > 1e-4


def test_zero_queries_give_zero_attention():
    """q = 0 makes every logit 0 and SiLU(0) = 0: the attention output vanishes and a one-layer model reduces to
    out-projection bias + feed-forward of the token itself, whatever the other tokens are."""
    shape = tiny_shape(L=1)
    w = synth.make_weights(shape, 21)
    d = shape.d_model
    wq = w.mat["w_qkv"].copy()
    wq[:, :d, :] = 0.0
    bq = w.vec["b_qkv"].copy()
    bq[:, :d] = 0.0
    m, _ = make_model(shape, 21, {"w_qkv": wq, "b_qkv": bq})
    rng = np.random.default_rng(3)
    p, s, c = ids(rng, 9), ids(rng, 2), ids(rng, 4)
    p2 = (p + 11) % 50
    assert np.max(np.abs(m.full(p, s, c) - m.full(p2, s, c))) <= 1e-12

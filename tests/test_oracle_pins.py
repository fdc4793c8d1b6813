"""Pins for the CPU checker (CPU only; run with -m "not gpu").

The paper prints no score for a worked example, so the checker is pinned by
(1) a dense-mask brute force written independently in numpy, (2) the textbook
causal special case against library attention, (3) the defining relation of
Section 2.3 (rank on cached prefix == full inference), (4) mask invariants
that follow from the item-independent prefix of Section 3.1, (5) Table 1's
KV footprint, and (6) planted mistakes that the pins must catch.
"""
import os

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2601_01712_b200 import synth
from tests import brute_force

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny_shape(L=2, d=16, H=2, F=32, vocab=50):
    return synth.ModelShape(L, d, H, d // H, F, vocab, synth.DTYPE_F32)


def make_model(shape, seed, params_override=None):
    w = synth.make_weights(shape, seed)
    params = {**w.mat, **w.vec}
    if params_override:
        params.update(params_override)
    m = ref.Model(shape.n_layers, shape.d_model, shape.n_heads, shape.d_head, shape.d_ff, shape.ln_eps, params)
    return m, params


def shape_dict(shape):
    return dict(n_layers=shape.n_layers, d_model=shape.d_model, n_heads=shape.n_heads, d_head=shape.d_head,
                ln_eps=shape.ln_eps)


def ids(rng, n, vocab=50):
    return rng.integers(0, vocab, n).astype(np.int32)


# ---------------------------------------------------------------- (1) brute force
@pytest.mark.parametrize("P,S,C", [(16, 4, 4), (9, 0, 3), (5, 3, 1), (1, 0, 1), (12, 4, 0), (7, 1, 5)])
def test_full_matches_dense_mask_brute_force(P, S, C):
    shape = tiny_shape()
    m, params = make_model(shape, 3)
    rng = np.random.default_rng(100 + P + S + C)
    p, s, c = ids(rng, P), ids(rng, S), ids(rng, C)
    got = m.full(p, s, c)
    want = brute_force.scores(shape_dict(shape), params, p, s, c)
    assert got.shape == (C,)
    if C:
        assert np.max(np.abs(got - want)) <= 1e-10


def test_brute_force_three_heads_one_layer():
    shape = synth.ModelShape(1, 24, 3, 8, 40, 50, synth.DTYPE_F32)
    m, params = make_model(shape, 4)
    rng = np.random.default_rng(7)
    p, s, c = ids(rng, 11), ids(rng, 2), ids(rng, 4)
    assert np.max(np.abs(m.full(p, s, c) - brute_force.scores(shape_dict(shape), params, p, s, c))) <= 1e-10


# ---------------------------------------------------------------- (2) textbook special case
def library_last_token_score(shape, params, ids_all, attn_mask=None):
    """A pre-LN transformer over one token sequence, written with torch's library routines and read at its
    last token.  attn_mask = None: ordinary causal attention (is_causal=True); else a boolean [T, T] mask."""
    t = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    d, H, dh = shape.d_model, shape.n_heads, shape.d_head
    x = t(params["emb"])[torch.tensor(np.asarray(ids_all).astype(np.int64))]
    T = x.shape[0]
    for l in range(shape.n_layers):
        a = torch.nn.functional.layer_norm(x, (d,), t(params["ln1_g"][l]), t(params["ln1_b"][l]), shape.ln_eps)
        qkv = torch.nn.functional.linear(a, t(params["w_qkv"][l]), t(params["b_qkv"][l]))
        q, k, v = [z.reshape(T, H, dh).transpose(0, 1) for z in qkv.split(d, dim=1)]
        if attn_mask is None:
            o = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)
        else:
            o = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=torch.tensor(attn_mask))
        o = o.transpose(0, 1).reshape(T, d)
        h = x + torch.nn.functional.linear(o, t(params["w_o"][l]), t(params["b_o"][l]))
        a2 = torch.nn.functional.layer_norm(h, (d,), t(params["ln2_g"][l]), t(params["ln2_b"][l]), shape.ln_eps)
        z = torch.nn.functional.silu(torch.nn.functional.linear(a2, t(params["w1"][l]), t(params["b1"][l])))
        x = h + torch.nn.functional.linear(z, t(params["w2"][l]), t(params["b2"][l]))
    a = torch.nn.functional.layer_norm(x[-1], (d,), t(params["lnf_g"]), t(params["lnf_b"]), shape.ln_eps)
    return float(a @ t(params["w_score"]) + float(params["b_score"][0]))


@pytest.mark.parametrize("P,S", [(13, 0), (9, 5), (1, 7), (6, 1)])
def test_causal_special_case_against_library_attention(P, S):
    """C = 1: [prefix; short-term; one candidate] is an ordinary causal sequence (every token sees exactly the
    tokens up to itself), so the candidate's score is a plain causal pre-LN transformer read at its last
    token.  With S > 0 this pins the short-term rows' causal edge, through every layer, against the library's
    own causal mask - a writing of the mask that shares nothing with the checker's or the brute force's."""
    shape = tiny_shape(L=2, d=16, H=2, F=32)
    m, params = make_model(shape, 5)
    rng = np.random.default_rng(11 + P + 31 * S)
    p, s, c = ids(rng, P), ids(rng, S), ids(rng, 1)
    got = m.full(p, s, c)[0]
    want = library_last_token_score(shape, params, np.concatenate([p, s, c]))
    assert abs(got - want) <= 1e-10
    K, V = m.preinfer(p)
    assert abs(m.rank_cached(K, V, s, c)[0] - want) <= 1e-10


@pytest.mark.parametrize("mistake", ["short_sees_later_short", "short_misses_itself", "short_misses_prefix"])
def test_library_pin_catches_a_wrong_short_term_edge(mistake):
    """The same library computation with the short-term rows' mask edge moved the way a plausible bug would
    move it: the candidate's score then differs from the checker's by far more than the pin's 1e-10, so a
    checker with that bug fails test_causal_special_case_against_library_attention."""
    shape = tiny_shape(L=2, d=16, H=2, F=32)
    m, params = make_model(shape, 5)
    rng = np.random.default_rng(12)
    P, S = 9, 5
    p, s, c = ids(rng, P), ids(rng, S), ids(rng, 1)
    T = P + S + 1
    mask = np.tril(np.ones((T, T), dtype=bool))
    assert abs(m.full(p, s, c)[0] - library_last_token_score(shape, params, np.concatenate([p, s, c]), mask)) <= 1e-10
    if mistake == "short_sees_later_short":
        mask[P:P + S, P:P + S] = True
    elif mistake == "short_misses_itself":
        mask[P:P + S, P:P + S] &= ~np.eye(S, dtype=bool)
    else:
        mask[P:P + S, :P] = False
    wrong = library_last_token_score(shape, params, np.concatenate([p, s, c]), mask)
    assert abs(m.full(p, s, c)[0] - wrong) > 1e-4


# ---------------------------------------------------------------- (3) defining relation
@pytest.mark.parametrize("P,S,C", [(16, 4, 4), (40, 0, 6), (33, 7, 1), (1, 2, 3)])
def test_rank_on_cached_prefix_equals_full_inference(P, S, C):
    shape = tiny_shape(L=3)
    m, _ = make_model(shape, 6)
    rng = np.random.default_rng(P * 31 + S)
    p, s, c = ids(rng, P), ids(rng, S), ids(rng, C)
    K, V = m.preinfer(p)
    assert K.shape == (3, P, shape.d_model)
    assert np.max(np.abs(m.rank_cached(K, V, s, c) - m.full(p, s, c))) <= 1e-10


def test_cached_equals_full_on_config1():
    wl = synth.workload(1)
    w = synth.make_weights(wl.model, wl.seed)
    sh = wl.model
    m = ref.Model(sh.n_layers, sh.d_model, sh.n_heads, sh.d_head, sh.d_ff, sh.ln_eps, {**w.mat, **w.vec})
    rng = np.random.default_rng(wl.seed)
    batch = synth.config1_batch(synth.ZipfIds(sh.vocab, wl.zipf_a), rng)
    assert batch.n_users == 4
    for i in range(batch.n_users):
        p, s, c = batch.user_slices(i)
        assert (len(p), len(s), len(c)) == (256, 32, 64)
        K, V = m.preinfer(p)
        a, b = m.rank_cached(K, V, s, c), m.full(p, s, c)
        assert np.max(np.abs(a - b)) <= 1e-9
        assert np.std(b) > 0.05          # scores are not degenerate


# ---------------------------------------------------------------- (4) invariants
def test_candidate_scores_do_not_depend_on_other_candidates():
    shape = tiny_shape()
    m, _ = make_model(shape, 8)
    rng = np.random.default_rng(21)
    p, s, c = ids(rng, 20), ids(rng, 5), ids(rng, 9)
    K, V = m.preinfer(p)
    all_scores = m.rank_cached(K, V, s, c)
    for i in (0, 4, 8):
        assert abs(m.rank_cached(K, V, s, c[i:i + 1])[0] - all_scores[i]) <= 1e-12
    perm = rng.permutation(len(c))
    assert np.max(np.abs(m.rank_cached(K, V, s, c[perm]) - all_scores[perm])) <= 1e-12
    assert np.max(np.abs(m.full(p, s, c[perm]) - m.full(p, s, c)[perm])) <= 1e-12


def test_short_term_tokens_are_causal_and_seen_by_candidates():
    shape = tiny_shape()
    m, _ = make_model(shape, 9)
    rng = np.random.default_rng(22)
    p, s, c = ids(rng, 12), ids(rng, 6), ids(rng, 3)
    base = m.full(p, s, c)
    s2 = s.copy()
    s2[-1] = (s2[-1] + 1) % 50
    assert np.max(np.abs(m.full(p, s2, c) - base)) > 1e-6      # candidates see every short-term token
    p2 = p.copy()
    p2[0] = (p2[0] + 1) % 50
    assert np.max(np.abs(m.full(p2, s, c) - base)) > 1e-6      # and the whole prefix


def test_prefix_kv_is_deterministic_causal_and_item_independent():
    shape = tiny_shape(L=2)
    m, _ = make_model(shape, 10)
    rng = np.random.default_rng(23)
    p = ids(rng, 24)
    K1, V1 = m.preinfer(p)
    K2, V2 = m.preinfer(p)
    assert np.array_equal(K1, K2) and np.array_equal(V1, V2)
    # changing prefix token i leaves rows < i untouched, in every layer
    i = 10
    q = p.copy()
    q[i] = (q[i] + 3) % 50
    K3, V3 = m.preinfer(q)
    assert np.array_equal(K1[:, :i], K3[:, :i]) and np.array_equal(V1[:, :i], V3[:, :i])
    assert np.max(np.abs(K1[:, i:] - K3[:, i:])) > 1e-6
    # a prefix of the prefix gives the same leading rows
    K4, V4 = m.preinfer(p[:15])
    assert np.max(np.abs(K4 - K1[:, :15])) <= 1e-12 and np.max(np.abs(V4 - V1[:, :15])) <= 1e-12
    # layer-0 keys are a function of the token alone: equal ids give equal rows
    p_same = np.full(6, 17, dtype=np.int32)
    K5, _ = m.preinfer(p_same)
    assert np.max(np.abs(K5[0] - K5[0][0])) <= 1e-12


def test_uniform_attention_when_keys_carry_no_signal():
    """With W_q = 0 and b_q = 0 every score is 0, softmax is uniform over the allowed set, and a
    candidate's attention output is the mean of the allowed V rows: checked through layer 0 by
    comparing with a model whose mask does not matter (all tokens equal)."""
    shape = tiny_shape(L=1)
    w = synth.make_weights(shape, 12)
    d = shape.d_model
    wq = w.mat["w_qkv"].copy()
    wq[:, :d, :] = 0.0
    bq = w.vec["b_qkv"].copy()
    bq[:, :d] = 0.0
    m, params = make_model(shape, 12, {"w_qkv": wq, "b_qkv": bq})
    rng = np.random.default_rng(24)
    p, s, c = ids(rng, 8), ids(rng, 2), ids(rng, 2)
    got = m.full(p, s, c)
    # closed form for one layer: o_c = mean over allowed keys of v_j
    f64 = lambda a: np.asarray(a, dtype=np.float64)
    ln = lambda z, g, b: (z - z.mean(-1, keepdims=True)) / np.sqrt(z.var(-1, keepdims=True) + shape.ln_eps) * g + b
    ids_all = np.concatenate([p, s, c])
    x = f64(params["emb"])[ids_all]
    a = ln(x, f64(params["ln1_g"][0]), f64(params["ln1_b"][0]))
    v = a @ f64(params["w_qkv"][0][2 * d:]).T + f64(params["b_qkv"][0][2 * d:])
    out = []
    for i in range(len(c)):
        t = len(p) + len(s) + i
        o = (v[:len(p) + len(s)].sum(0) + v[t]) / (len(p) + len(s) + 1)
        h = x[t] + o @ f64(params["w_o"][0]).T + f64(params["b_o"][0])
        z = ln(h, f64(params["ln2_g"][0]), f64(params["ln2_b"][0])) @ f64(params["w1"][0]).T + f64(params["b1"][0])
        xx = h + (z / (1 + np.exp(-z))) @ f64(params["w2"][0]).T + f64(params["b2"][0])
        out.append(ln(xx, f64(params["lnf_g"]), f64(params["lnf_b"])) @ f64(params["w_score"]) + params["b_score"][0])
    assert np.max(np.abs(got - np.array(out))) <= 1e-10


def test_batch_equals_single_user_calls():
    shape = tiny_shape()
    m, _ = make_model(shape, 13)
    rng = np.random.default_rng(25)
    zipf = synth.ZipfIds(shape.vocab, 1.1)
    b = synth.make_batch(zipf, rng, [9, 17, 5], [2, 0, 3], [4, 1, 2])
    for i in range(3):
        p, s, c = b.user_slices(i)
        K, V = m.preinfer(p)
        assert np.max(np.abs(m.rank_cached(K, V, s, c) - m.full(p, s, c))) <= 1e-10


# ---------------------------------------------------------------- (5) closed forms the paper prints
def test_kv_footprint_matches_table1():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table1_kv_cache.txt")) if not l.startswith("#")]
    seq, layers, esize, dim, size = map(int, rows[0])
    assert ref.kv_bytes(seq, layers, dim, esize) == size == 32 * 1024 * 1024
    shape = synth.ModelShape(layers, dim, 4, 64, 1024, 10, synth.DTYPE_F32)
    assert shape.kv_bytes(seq) == size
    m, _ = make_model(synth.ModelShape(8, 16, 2, 8, 32, 50, synth.DTYPE_F32), 1)
    K, V = m.preinfer(np.arange(10, dtype=np.int32))
    assert K.size + V.size == 10 * 8 * 2 * 16


# ---------------------------------------------------------------- (6) planted mistakes are caught
@pytest.mark.parametrize("mistake", ["candidates_see_each_other", "strict_causal", "no_sqrt_scale", "drop_bias"])
def test_pins_catch_planted_mistakes(mistake):
    """The brute force is perturbed the way a plausible bug would perturb the checker; the
    comparison used above must then fail, i.e. the pin has teeth."""
    shape = tiny_shape()
    m, params = make_model(shape, 14)
    rng = np.random.default_rng(26)
    p, s, c = ids(rng, 10), ids(rng, 3), ids(rng, 4)
    got = m.full(p, s, c)
    sd = shape_dict(shape)
    P, S, C = len(p), len(s), len(c)
    mask = brute_force.dense_mask(P, S, C)
    w2 = dict(params)
    if mistake == "candidates_see_each_other":
        mask = np.tril(np.ones_like(mask))
    elif mistake == "strict_causal":
        mask = mask & ~np.eye(P + S + C, dtype=bool)
        mask[0, 0] = True
    elif mistake == "no_sqrt_scale":
        # scaling the query projection by sqrt(d_h) is the same as forgetting the 1/sqrt(d_h)
        d = shape.d_model
        wq, bq = params["w_qkv"].copy(), params["b_qkv"].copy()
        wq[:, :d, :] *= np.sqrt(shape.d_head)
        bq[:, :d] *= np.sqrt(shape.d_head)
        w2["w_qkv"], w2["b_qkv"] = wq, bq
    elif mistake == "drop_bias":
        w2["b_qkv"] = np.zeros_like(params["b_qkv"])
    ids_all = np.concatenate([p, s, c]).astype(np.int64)
    x = brute_force.forward(sd, w2, ids_all, mask)[P + S:]
    ln = lambda z, g, b: (z - z.mean(-1, keepdims=True)) / np.sqrt(z.var(-1, keepdims=True) + shape.ln_eps) * g + b
    wrong = ln(x, params["lnf_g"].astype(np.float64), params["lnf_b"].astype(np.float64)) @ params["w_score"].astype(np.float64)
    assert np.max(np.abs(got - wrong)) > 1e-4


# ---------------------------------------------------------------- the bf16 noise yardstick of the GPU tests
def test_noise_emulation_without_rounding_is_the_model_and_rounding_adds_small_noise():
    from tests import bf16_noise
    shape = synth.ModelShape(2, 128, 2, 64, 256, 300, synth.DTYPE_BF16)
    w = synth.make_weights(shape, 15)
    params = {**w.mat, **w.vec}
    m = ref.Model(shape.n_layers, shape.d_model, shape.n_heads, shape.d_head, shape.d_ff, shape.ln_eps, params)
    rng = np.random.default_rng(27)
    p, s, c = ids(rng, 70, 300), ids(rng, 9, 300), ids(rng, 40, 300)
    sd = dict(shape_dict(shape), attn_kind=0)
    want = m.full(p, s, c)
    assert np.max(np.abs(bf16_noise.scores(sd, params, p, s, c, sites=()) - want)) <= 1e-9
    noisy = bf16_noise.scores(sd, params, p, s, c)
    rms = float(np.sqrt(np.mean((noisy - want) ** 2)))
    assert 5e-4 < rms < 1e-2                                    # every site rounded: small, not zero
    for site in bf16_noise.SITES:                               # each site alone moves the scores, by less than all together would at worst
        e = bf16_noise.scores(sd, params, p, s, c, sites=(site,)) - want
        assert 0 < float(np.max(np.abs(e))) < 2e-2
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.1415927, 1e-30, -65504.0])
    assert np.array_equal(bf16_noise.bf16(x).astype(np.float32), torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).float().numpy())
    # the pointwise variant
    m1 = ref.Model(shape.n_layers, shape.d_model, shape.n_heads, shape.d_head, shape.d_ff, shape.ln_eps, params, attn_kind=1)
    sd1 = dict(shape_dict(shape), attn_kind=1)
    assert np.max(np.abs(bf16_noise.scores(sd1, params, p, s, c, sites=()) - m1.full(p, s, c))) <= 1e-9


# ---------------------------------------------------------------- input recipe
def test_zipf_ids_are_seeded_in_range_and_skewed():
    z = synth.ZipfIds(10_000, 1.1)
    a = z.draw(np.random.default_rng(1), 20000)
    b = z.draw(np.random.default_rng(1), 20000)
    assert np.array_equal(a, b) and a.dtype == np.int32 and a.min() >= 0 and a.max() < 10_000
    top = np.bincount(a, minlength=10_000).max() / len(a)
    assert 0.08 < top < 0.2                       # rank-1 mass of Zipf(1.1) over 10k is about 0.12
    ranks = np.arange(10_000, dtype=np.int64)
    assert len(np.unique((ranks * synth.ZipfIds.MULT) % 10_000)) == 10_000
    r = np.arange(1_000_000, dtype=np.int64)
    assert len(np.unique((r * synth.ZipfIds.MULT) % 1_000_000)) == 1_000_000


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.1415927], dtype=np.float32)
    bits = synth.round_to_bf16_bits(x)
    want = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    assert np.array_equal(synth.bf16_bits_to_f32(bits), torch.tensor(x).to(torch.bfloat16).float().numpy())

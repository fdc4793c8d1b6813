"""Dense-mask brute force of the ranking model in numpy (fp64).

A second, independent writing of the model used only to pin the CPU checker on
tiny inputs: it materialises the full (P+S+C)^2 boolean mask and evaluates
softmax(Q K^T / sqrt(d_h) + mask) V head by head - or, for the pointwise
variant (``shape["attn_kind"] == 1``), (SiLU(Q K^T / sqrt(d_h)) * mask) V divided
by each row's count of visible keys.  It shares no code with the checker in
``oracle/`` or with the CUDA library.
"""
import numpy as np


def dense_mask(P, S, C):
    """mask[t, j] is True where query t may look at key j (Section 3.1: the
    prefix is item-independent; candidates see prefix, short-term and self)."""
    T = P + S + C
    m = np.zeros((T, T), dtype=bool)
    for t in range(T):
        for j in range(T):
            if t < P + S:
                m[t, j] = j <= t
            else:
                m[t, j] = (j < P + S) or (j == t)
    return m


def _ln(z, g, b, eps):
    mu = z.mean(axis=-1, keepdims=True)
    var = ((z - mu) ** 2).mean(axis=-1, keepdims=True)
    return (z - mu) / np.sqrt(var + eps) * g + b


def forward(shape, w, ids_all, mask):
    """Hidden states after all layers for tokens ``ids_all`` under ``mask``.
    ``w`` maps names to fp32 arrays, linear weights [L, out, in]."""
    L, d, H, dh = shape["n_layers"], shape["d_model"], shape["n_heads"], shape["d_head"]
    eps = shape["ln_eps"]
    f = lambda name, l: np.asarray(w[name][l], dtype=np.float64)
    x = np.asarray(w["emb"], dtype=np.float64)[np.asarray(ids_all)]
    T = x.shape[0]
    for l in range(L):
        a = _ln(x, f("ln1_g", l), f("ln1_b", l), eps)
        qkv = a @ f("w_qkv", l).T + f("b_qkv", l)
        q, k, v = qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]
        att = np.zeros((T, d))
        for h in range(H):
            sl = slice(h * dh, (h + 1) * dh)
            s = q[:, sl] @ k[:, sl].T / np.sqrt(dh)
            if shape.get("attn_kind", 0) == 1:
                p = np.where(mask, s / (1.0 + np.exp(-s)), 0.0)
                att[:, sl] = (p @ v[:, sl]) / mask.sum(axis=1, keepdims=True)
                continue
            s = np.where(mask, s, -np.inf)
            s = s - s.max(axis=1, keepdims=True)
            p = np.exp(s)
            p = p / p.sum(axis=1, keepdims=True)
            att[:, sl] = p @ v[:, sl]
        hmid = x + att @ f("w_o", l).T + f("b_o", l)
        a2 = _ln(hmid, f("ln2_g", l), f("ln2_b", l), eps)
        z = a2 @ f("w1", l).T + f("b1", l)
        z = z / (1.0 + np.exp(-z))
        x = hmid + z @ f("w2", l).T + f("b2", l)
    return x


def scores(shape, w, prefix_ids, short_ids, cand_ids):
    P, S, C = len(prefix_ids), len(short_ids), len(cand_ids)
    ids = np.concatenate([np.asarray(prefix_ids, dtype=np.int64), np.asarray(short_ids, dtype=np.int64),
                          np.asarray(cand_ids, dtype=np.int64)])
    x = forward(shape, w, ids, dense_mask(P, S, C))
    xc = x[P + S:]
    a = _ln(xc, np.asarray(w["lnf_g"], dtype=np.float64), np.asarray(w["lnf_b"], dtype=np.float64), shape["ln_eps"])
    return a @ np.asarray(w["w_score"], dtype=np.float64) + float(w["b_score"][0])

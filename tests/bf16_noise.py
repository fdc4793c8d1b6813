"""How large must the score error of a bf16 model be?  A numpy (fp64) writing of the ranking model that rounds to bf16 at
chosen sites - the places where a bf16 tensor-core implementation has no choice, because the value is an operand of a
bf16 matrix product:

    a     LayerNorm-1 output            (A operand of the QKV projection)
    qkv   projected queries, keys and values (operands of Q K^T and P V; K and V are also what the pages store)
    p     the unnormalised attention weights (A operand of P V; the row sum is taken before the rounding)
    att   the attention output          (A operand of the output projection)
    a2    LayerNorm-2 output            (A operand of the first feed-forward product)
    hid   SiLU hidden activations       (A operand of the second feed-forward product)

Everything else (accumulation, residual stream, LayerNorm statistics, softmax state, scoring head) stays in full
precision.  With no site rounded this is the model itself (it then agrees with the checker to 1e-9); with all of them
rounded it is one *sample* of the rounding noise that any bf16 implementation of this shape produces: not the same
numbers as another implementation (rounding decisions flip on the last bit of their inputs), but the same distribution.
The parity tests use its root-mean-square error as the yardstick for shapes other than the named workloads.

Test infrastructure: shares no code with the checker in ``oracle/`` or with the CUDA library.
"""
import numpy as np

SITES = ("a", "qkv", "p", "att", "a2", "hid")


def bf16(x):
    """Round fp64 values to the nearest bf16 (ties to even), returned as fp64."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


def _ln(z, g, b, eps):
    mu = z.mean(axis=-1, keepdims=True)
    var = ((z - mu) ** 2).mean(axis=-1, keepdims=True)
    return (z - mu) / np.sqrt(var + eps) * g + b


def _mask(P, S, C):
    T = P + S + C
    t = np.arange(T)[:, None]
    j = np.arange(T)[None, :]
    return np.where(t < P + S, j <= t, (j < P + S) | (j == t))


def scores(shape, w, prefix_ids, short_ids, cand_ids, sites=SITES):
    """Scores of the candidates with bf16 rounding at ``sites`` (a subset of SITES).  shape: n_layers, d_model, n_heads,
    d_head, ln_eps, attn_kind; w: name -> fp32 array, linear weights [L, out, in]."""
    rd = lambda name, x: bf16(x) if name in sites else x
    L, d, H, dh, eps = shape["n_layers"], shape["d_model"], shape["n_heads"], shape["d_head"], shape["ln_eps"]
    kind = shape.get("attn_kind", 0)
    P, S, C = len(prefix_ids), len(short_ids), len(cand_ids)
    ids = np.concatenate([np.asarray(prefix_ids, np.int64), np.asarray(short_ids, np.int64), np.asarray(cand_ids, np.int64)])
    f = lambda name, l: np.asarray(w[name][l], dtype=np.float64)
    x = np.asarray(w["emb"], dtype=np.float64)[ids]
    mask = _mask(P, S, C)
    n_seen = mask.sum(axis=1, keepdims=True)
    T = P + S + C
    for l in range(L):
        a = rd("a", _ln(x, f("ln1_g", l), f("ln1_b", l), eps))
        qkv = rd("qkv", a @ f("w_qkv", l).T + f("b_qkv", l))
        q, k, v = qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]
        att = np.zeros((T, d))
        for h in range(H):
            sl = slice(h * dh, (h + 1) * dh)
            s = q[:, sl] @ k[:, sl].T / np.sqrt(dh)
            if kind == 1:
                pw = np.where(mask, s / (1.0 + np.exp(-s)), 0.0)
                att[:, sl] = (rd("p", pw) @ v[:, sl]) / n_seen
            else:
                s = np.where(mask, s, -np.inf)
                pw = np.exp(s - s.max(axis=1, keepdims=True))
                att[:, sl] = (rd("p", pw) @ v[:, sl]) / pw.sum(axis=1, keepdims=True)
        att = rd("att", att)
        mid = x + att @ f("w_o", l).T + f("b_o", l)
        a2 = rd("a2", _ln(mid, f("ln2_g", l), f("ln2_b", l), eps))
        z = a2 @ f("w1", l).T + f("b1", l)
        x = mid + rd("hid", z / (1.0 + np.exp(-z))) @ f("w2", l).T + f("b2", l)
    xc = x[P + S:]
    af = _ln(xc, np.asarray(w["lnf_g"], np.float64), np.asarray(w["lnf_b"], np.float64), eps)
    return af @ np.asarray(w["w_score"], np.float64) + float(w["b_score"][0])

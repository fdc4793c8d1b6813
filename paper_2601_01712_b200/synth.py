"""Seeded synthetic inputs for the relay-race GR inference path.

This module only *draws* inputs (model shapes, random weights, item ids,
sequence lengths, page permutations).  It holds none of the model's
arithmetic: both the CUDA path and the CPU checker consume what it returns.

The production queries the paper evaluates on are proprietary; these inputs
stand in for them with the shapes the paper states for its workloads
(Section 4.1: 1K to tens of thousands of tokens, dims 128-1024, several to
tens of layers; Section 4.4: about 512 candidate items per query).

Conventions
-----------
* Linear weights use the ``[out, in]`` row-major layout (``y = x @ W.T + b``).
* Matrices and the embedding table are generated in fp32 and, for a bf16
  model, rounded once to bf16 (round-to-nearest-even).  ``*_f32`` views hold
  the rounded values widened back to fp32, so a checker reads exactly the
  numbers the device reads.
* Vectors (LayerNorm gains/biases, linear biases, scoring vector) stay fp32.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

DTYPE_F32 = 0
DTYPE_BF16 = 1
PAGE_TOKENS = 64
BASE_SEED = 17120


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_heads: int
    d_head: int
    d_ff: int
    vocab: int
    dtype: int
    ln_eps: float = 1e-5
    page_tokens: int = PAGE_TOKENS
    attn_kind: int = 0            # 0 softmax attention, 1 pointwise SiLU attention (HSTU style)

    def kv_bytes(self, prefix_len: int) -> int:
        """Bytes of per-layer K and V kept for a prefix of ``prefix_len`` tokens."""
        esize = 4 if self.dtype == DTYPE_F32 else 2
        return prefix_len * self.n_layers * 2 * self.d_model * esize


MODEL_TINY = ModelShape(2, 64, 2, 32, 256, 10_000, DTYPE_F32)
MODEL_PROD = ModelShape(4, 256, 4, 64, 1024, 1_000_000, DTYPE_BF16)
MODEL_LONG = ModelShape(8, 512, 8, 64, 2048, 1_000_000, DTYPE_BF16)


def round_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 array -> uint16 array of bf16 bit patterns, round-to-nearest-even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Weights:
    """Random-initialised parameters of one model.

    ``mat[name]`` is the fp32 value every consumer must use (already rounded to
    bf16 precision for a bf16 model); ``bits[name]`` is the uint16 bf16 pattern
    (bf16 models only); ``vec[name]`` are fp32 vectors.
    """
    shape: ModelShape
    mat: Dict[str, np.ndarray] = field(default_factory=dict)
    bits: Dict[str, np.ndarray] = field(default_factory=dict)
    vec: Dict[str, np.ndarray] = field(default_factory=dict)


def make_weights(shape: ModelShape, seed: int, vocab: Optional[int] = None) -> Weights:
    """Embeddings N(0, 1/sqrt(d)) (std), matrices N(0, 1/sqrt(fan_in)), biases
    N(0, 0.02), LayerNorm gains 1 + 0.1 N(0,1), LayerNorm biases 0.1 N(0,1),
    scoring vector N(0, 1/sqrt(d)), scoring bias 0."""
    rng = np.random.default_rng(seed)
    L, d, F = shape.n_layers, shape.d_model, shape.d_ff
    V = shape.vocab if vocab is None else vocab
    w = Weights(shape)

    def matrix(name, dims, std):
        a = rng.standard_normal(dims, dtype=np.float32) * np.float32(std)
        if shape.dtype == DTYPE_BF16:
            b = round_to_bf16_bits(a)
            w.bits[name] = b
            a = bf16_bits_to_f32(b)
        w.mat[name] = a

    def vector(name, dims, mean, std):
        w.vec[name] = (np.float32(mean) + rng.standard_normal(dims, dtype=np.float32) * np.float32(std))

    matrix("emb", (V, d), 1.0 / np.sqrt(d))
    matrix("w_qkv", (L, 3 * d, d), 1.0 / np.sqrt(d))
    matrix("w_o", (L, d, d), 1.0 / np.sqrt(d))
    matrix("w1", (L, F, d), 1.0 / np.sqrt(d))
    matrix("w2", (L, d, F), 1.0 / np.sqrt(F))
    vector("ln1_g", (L, d), 1.0, 0.1)
    vector("ln1_b", (L, d), 0.0, 0.1)
    vector("ln2_g", (L, d), 1.0, 0.1)
    vector("ln2_b", (L, d), 0.0, 0.1)
    vector("b_qkv", (L, 3 * d), 0.0, 0.02)
    vector("b_o", (L, d), 0.0, 0.02)
    vector("b1", (L, F), 0.0, 0.02)
    vector("b2", (L, d), 0.0, 0.02)
    vector("lnf_g", (d,), 1.0, 0.1)
    vector("lnf_b", (d,), 0.0, 0.1)
    vector("w_score", (d,), 0.0, 1.0 / np.sqrt(d))
    w.vec["b_score"] = np.zeros((1,), dtype=np.float32)
    return w


class ZipfIds:
    """Item ids with rank r in 1..V drawn with p(r) proportional to r^-a by
    inverse CDF on a float64 cumulative table; the rank is scattered over the
    id space by id = ((r-1) * 2654435761) mod V (a bijection whenever V is
    coprime to the prime multiplier), so hot rows are not adjacent."""

    MULT = 2654435761

    def __init__(self, vocab: int, a: float):
        self.vocab = int(vocab)
        p = np.arange(1, self.vocab + 1, dtype=np.float64) ** (-float(a))
        self.cdf = np.cumsum(p)
        self.cdf /= self.cdf[-1]

    def draw(self, rng: np.random.Generator, n: int) -> np.ndarray:
        u = rng.random(n)
        r = np.searchsorted(self.cdf, u, side="left").astype(np.int64)
        r = np.minimum(r, self.vocab - 1)
        return ((r * self.MULT) % self.vocab).astype(np.int32)


@dataclass
class Batch:
    """One jagged batch: flat id arrays and ``n_users + 1`` offsets each."""
    users: np.ndarray          # uint64 [B]
    prefix_ids: np.ndarray     # int32 [sum P]
    prefix_off: np.ndarray     # int32 [B+1]
    short_ids: np.ndarray
    short_off: np.ndarray
    cand_ids: np.ndarray
    cand_off: np.ndarray

    @property
    def n_users(self) -> int:
        return int(self.users.shape[0])

    def user_slices(self, i: int):
        p = self.prefix_ids[self.prefix_off[i]:self.prefix_off[i + 1]]
        s = self.short_ids[self.short_off[i]:self.short_off[i + 1]]
        c = self.cand_ids[self.cand_off[i]:self.cand_off[i + 1]]
        return p, s, c


def _offsets(lengths) -> np.ndarray:
    off = np.zeros(len(lengths) + 1, dtype=np.int64)
    np.cumsum(np.asarray(lengths, dtype=np.int64), out=off[1:])
    assert off[-1] < 2 ** 31
    return off.astype(np.int32)


def make_batch(zipf: ZipfIds, rng: np.random.Generator, p_lens, s_lens, c_lens,
               first_user: int = 0) -> Batch:
    B = len(p_lens)
    assert len(s_lens) == B and len(c_lens) == B
    users = (np.arange(B, dtype=np.uint64) + np.uint64(first_user))
    po, so, co = _offsets(p_lens), _offsets(s_lens), _offsets(c_lens)
    return Batch(users,
                 zipf.draw(rng, int(po[-1])), po,
                 zipf.draw(rng, int(so[-1])), so,
                 zipf.draw(rng, int(co[-1])), co)


def draw_short_cand(zipf: ZipfIds, rng: np.random.Generator, batch: Batch) -> Batch:
    """Same users and prefixes, fresh short-term and candidate ids (same lengths)."""
    return Batch(batch.users, batch.prefix_ids, batch.prefix_off,
                 zipf.draw(rng, int(batch.short_off[-1])), batch.short_off,
                 zipf.draw(rng, int(batch.cand_off[-1])), batch.cand_off)


def log_uniform_int(rng: np.random.Generator, lo: int, hi: int, n: int) -> np.ndarray:
    return np.rint(np.exp(rng.uniform(np.log(lo), np.log(hi), n))).astype(np.int64)


def shuffled_pages(rng: np.random.Generator, n_pages_total: int, counts) -> List[np.ndarray]:
    """A seeded shuffle of the pool's page ids dealt out to users: user i gets
    ``counts[i]`` distinct pages, scattered over the whole slab."""
    perm = rng.permutation(n_pages_total).astype(np.int32)
    out, at = [], 0
    for c in counts:
        out.append(perm[at:at + int(c)].copy())
        at += int(c)
    assert at <= n_pages_total
    return out


def pages_for(prefix_len: int, page_tokens: int = PAGE_TOKENS) -> int:
    return (int(prefix_len) + page_tokens - 1) // page_tokens


@dataclass(frozen=True)
class Workload:
    name: str
    model: ModelShape
    seed: int
    zipf_a: float


def workload(index: int) -> Workload:
    """The five evaluation configurations (index 1..5)."""
    table = {
        1: ("tiny_fp32", MODEL_TINY),
        2: ("prod_rank_bf16", MODEL_PROD),
        3: ("jagged_bf16", MODEL_PROD),
        4: ("long_seq_bf16", MODEL_LONG),
        5: ("reload_tier_bf16", MODEL_PROD),
    }
    name, model = table[index]
    return Workload(name, model, BASE_SEED + index, 1.1)


def config1_batch(zipf, rng) -> Batch:
    return make_batch(zipf, rng, [256] * 4, [32] * 4, [64] * 4)


def config2_batch(zipf, rng, n_users: int = 32, prefix: int = 2048) -> Batch:
    return make_batch(zipf, rng, [prefix] * n_users, [64] * n_users, [512] * n_users)


def config3_lengths(rng, n_users: int = 128):
    p = log_uniform_int(rng, 512, 8192, n_users)
    s = rng.integers(16, 128, n_users, endpoint=True)
    c = rng.integers(128, 1024, n_users, endpoint=True)
    return p, s, c


def config4_batch(zipf, rng, prefix: int, n_users: int = 16) -> Batch:
    return make_batch(zipf, rng, [prefix] * n_users, [128] * n_users, [1024] * n_users)

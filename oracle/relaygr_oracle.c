/*
 * CPU checker for relay-race GR inference.  TEST INFRASTRUCTURE ONLY: nothing
 * on the product path may call, link or import this file.  It shares no code
 * with the CUDA library.
 *
 * What it computes (all arithmetic in fp64; parameters arrive as fp32 values
 * and are widened on read):
 *
 *   The ranking model f of Section 2.3 is a stack of pre-LayerNorm transformer
 *   blocks with softmax attention, a two-matrix SiLU feed-forward net, a final
 *   LayerNorm and a linear head giving one logit per candidate item.  (The
 *   paper never prints the block equations; this block is the one the
 *   evaluation configurations name.)
 *
 *   A user's tokens, in order: P long-term prefix tokens, S short-term tokens,
 *   C candidate items.  Query t may attend to key j iff
 *       t in prefix     : j <= t
 *       t in short-term : j <= t                (whole prefix + earlier short)
 *       t is a candidate: j < P+S  or  j == t   (prefix, short-term, itself)
 *   so the prefix is item-independent (Section 3.1) and candidates never see
 *   one another.
 *
 *   attn_kind selects how the allowed keys are aggregated:
 *     0  softmax attention      o_t = sum_j softmax_j(q_t.k_j / sqrt(dh)) v_j
 *     1  pointwise aggregated attention in the style of HSTU, the model family
 *        the paper's evaluation names (Section 5.1): the softmax is replaced by
 *        an elementwise SiLU, o_t = (1 / |A(t)|) sum_j SiLU(q_t.k_j / sqrt(dh)) v_j.
 *        Readings: HSTU's relative attention bias is left out (no positions or
 *        timestamps exist in this model), the logit scale 1/sqrt(dh) is kept
 *        from the softmax block, and the normaliser is the number of keys the
 *        query may see (HSTU divides by the sequence length).  Only the
 *        attention changes; the block around it stays the pre-LN transformer.
 *
 *   orc_full        f([U,S_l,S~_l,I], {})  - one pass over all P+S+C tokens.
 *   orc_preinfer    psi <- f([U,S_l,{},{}], {}) - prefix only, returns the
 *                   per-layer K and V rows (Section 2.3, Section 4.1 "cache
 *                   semantics").
 *   orc_rank_cached f([{},{},S~_l,I], psi) - S+C tokens whose keys are the
 *                   cached prefix rows followed by their own.
 *
 * The relation |full - rank_cached| <= eps of Section 2.3 holds exactly here
 * (up to rounding order) because no prefix token attends outside the prefix.
 *
 * No tiling, blocking, fusion or caching beyond that definition.  OpenMP only
 * spreads independent rows over cores.
 *
 * Pins (tests, CPU only): dense-mask brute force in numpy on tiny inputs, the
 * causal special case against library attention, cached == full, mask
 * invariants, Table 1's 32 MB footprint.  No score value is printed in the
 * paper, so scores are pinned by those alone.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, d_model, n_heads, d_head, d_ff;
    double ln_eps;
    int32_t attn_kind;                              /* 0 softmax, 1 pointwise SiLU (see above) */
} orc_cfg;

/* Linear weights are [out, in] row-major: y = x W^T + b. */
typedef struct {
    const float *emb;                               /* [vocab, d] */
    const float *ln1_g, *ln1_b, *ln2_g, *ln2_b;     /* [L, d] */
    const float *w_qkv, *b_qkv;                     /* [L, 3d, d], [L, 3d] */
    const float *w_o, *b_o;                         /* [L, d, d], [L, d] */
    const float *w1, *b1;                           /* [L, F, d], [L, F] */
    const float *w2, *b2;                           /* [L, d, F], [L, d] */
    const float *lnf_g, *lnf_b, *w_score, *b_score; /* [d], [d], [d], [1] */
} orc_weights;

/* LN(z) = (z - mean) / sqrt(var + eps) * g + b, biased variance over d. */
static void layer_norm(const double *z, const float *g, const float *b, double eps, int d, double *out)
{
    double mean = 0.0, var = 0.0;
    for (int i = 0; i < d; ++i) mean += z[i];
    mean /= d;
    for (int i = 0; i < d; ++i) var += (z[i] - mean) * (z[i] - mean);
    var /= d;
    double rstd = 1.0 / sqrt(var + eps);
    for (int i = 0; i < d; ++i) out[i] = (z[i] - mean) * rstd * (double)g[i] + (double)b[i];
}

/* y[n] = sum_k a[k] W[n][k] + bias[n] */
static void linear(const double *a, const float *W, const float *bias, int n_in, int n_out, double *y)
{
    for (int n = 0; n < n_out; ++n) {
        const float *w = W + (size_t)n * n_in;
        double acc = 0.0;
#pragma omp simd reduction(+ : acc)
        for (int k = 0; k < n_in; ++k) acc += a[k] * (double)w[k];
        y[n] = acc + (bias ? (double)bias[n] : 0.0);
    }
}

static double silu(double z) { return z / (1.0 + exp(-z)); }

/* The attention mask on global positions (prefix [0,P), short [P,P+S), candidates after). */
static int allowed(int64_t P, int64_t S, int64_t t, int64_t j)
{
    if (t < P + S) return j <= t;
    return j < P + S || j == t;
}

/*
 * One block over n tokens at global positions pos0 .. pos0+n-1.  Keys/values
 * visible to them: n_ctx cached rows at positions 0 .. n_ctx-1 (Kctx, Vctx,
 * [n_ctx, d]) followed by the rows of these n tokens (positions pos0 ...).
 * x [n, d] is updated in place.  If Kout/Vout are given, the K and V rows of
 * the n tokens are copied out.
 */
static void block(const orc_cfg *c, const orc_weights *w, int l, int64_t P, int64_t S,
                  int64_t n, int64_t pos0, double *x,
                  int64_t n_ctx, const double *Kctx, const double *Vctx,
                  double *Kout, double *Vout)
{
    const int d = c->d_model, H = c->n_heads, dh = c->d_head, F = c->d_ff;
    const float *g1 = w->ln1_g + (size_t)l * d, *be1 = w->ln1_b + (size_t)l * d;
    const float *g2 = w->ln2_g + (size_t)l * d, *be2 = w->ln2_b + (size_t)l * d;
    const float *Wqkv = w->w_qkv + (size_t)l * 3 * d * d, *bqkv = w->b_qkv ? w->b_qkv + (size_t)l * 3 * d : NULL;
    const float *Wo = w->w_o + (size_t)l * d * d, *bo = w->b_o ? w->b_o + (size_t)l * d : NULL;
    const float *W1 = w->w1 + (size_t)l * F * d, *b1 = w->b1 ? w->b1 + (size_t)l * F : NULL;
    const float *W2 = w->w2 + (size_t)l * d * F, *b2 = w->b2 ? w->b2 + (size_t)l * d : NULL;

    double *qkv = (double *)malloc(sizeof(double) * (size_t)n * 3 * d);
    double *att = (double *)malloc(sizeof(double) * (size_t)n * d);

    /* a = LN1(x); [q|k|v] = a Wqkv^T + b */
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n; ++t) {
        double a[d];
        layer_norm(x + t * d, g1, be1, c->ln_eps, d, a);
        linear(a, Wqkv, bqkv, d, 3 * d, qkv + t * 3 * d);
    }
    if (Kout && Vout) {
        for (int64_t t = 0; t < n; ++t) {
            memcpy(Kout + t * d, qkv + t * 3 * d + d, sizeof(double) * d);
            memcpy(Vout + t * d, qkv + t * 3 * d + 2 * d, sizeof(double) * d);
        }
    }

    /* o_t = sum_{j in A(t)} softmax_j(q_t . k_j / sqrt(dh)) v_j, per head;
     * or, attn_kind 1, o_t = (1 / |A(t)|) sum_{j in A(t)} SiLU(q_t . k_j / sqrt(dh)) v_j */
    const double scale = 1.0 / sqrt((double)dh);
    const int64_t n_keys = n_ctx + n;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t t = 0; t < n; ++t) {
        double *s = (double *)malloc(sizeof(double) * (size_t)n_keys);
        const int64_t tpos = pos0 + t;
        for (int h = 0; h < H; ++h) {
            const double *q = qkv + t * 3 * d + h * dh;
            if (c->attn_kind == 1) {
                double *o = att + t * d + h * dh;
                for (int e = 0; e < dh; ++e) o[e] = 0.0;
                int64_t n_seen = 0;
                for (int64_t j = 0; j < n_keys; ++j) {
                    const int64_t jpos = j < n_ctx ? j : pos0 + (j - n_ctx);
                    if (!allowed(P, S, tpos, jpos)) continue;
                    const double *k = j < n_ctx ? Kctx + j * d + h * dh : qkv + (j - n_ctx) * 3 * d + d + h * dh;
                    const double *v = j < n_ctx ? Vctx + j * d + h * dh : qkv + (j - n_ctx) * 3 * d + 2 * d + h * dh;
                    double dot = 0.0;
                    for (int e = 0; e < dh; ++e) dot += q[e] * k[e];
                    const double p = silu(dot * scale);
                    for (int e = 0; e < dh; ++e) o[e] += p * v[e];
                    ++n_seen;
                }
                for (int e = 0; e < dh; ++e) o[e] /= (double)n_seen;     /* a query always sees itself */
                continue;
            }
            double m = -INFINITY;
            for (int64_t j = 0; j < n_keys; ++j) {
                const int64_t jpos = j < n_ctx ? j : pos0 + (j - n_ctx);
                if (!allowed(P, S, tpos, jpos)) { s[j] = -INFINITY; continue; }
                const double *k = j < n_ctx ? Kctx + j * d + h * dh : qkv + (j - n_ctx) * 3 * d + d + h * dh;
                double dot = 0.0;
                for (int e = 0; e < dh; ++e) dot += q[e] * k[e];
                s[j] = dot * scale;
                if (s[j] > m) m = s[j];
            }
            double denom = 0.0;
            for (int64_t j = 0; j < n_keys; ++j) {
                s[j] = (s[j] == -INFINITY) ? 0.0 : exp(s[j] - m);
                denom += s[j];
            }
            double *o = att + t * d + h * dh;
            for (int e = 0; e < dh; ++e) o[e] = 0.0;
            for (int64_t j = 0; j < n_keys; ++j) {
                if (s[j] == 0.0) continue;
                const double *v = j < n_ctx ? Vctx + j * d + h * dh : qkv + (j - n_ctx) * 3 * d + 2 * d + h * dh;
                const double p = s[j] / denom;
                for (int e = 0; e < dh; ++e) o[e] += p * v[e];
            }
        }
        free(s);
    }

    /* h = x + o Wo^T + bo ;  x <- h + W2 SiLU(W1 LN2(h) + b1) + b2 */
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n; ++t) {
        double proj[d], a[d], hid[F], out[d];
        double *xt = x + t * d;
        linear(att + t * d, Wo, bo, d, d, proj);
        for (int i = 0; i < d; ++i) xt[i] += proj[i];
        layer_norm(xt, g2, be2, c->ln_eps, d, a);
        linear(a, W1, b1, d, F, hid);
        for (int i = 0; i < F; ++i) hid[i] = silu(hid[i]);
        linear(hid, W2, b2, F, d, out);
        for (int i = 0; i < d; ++i) xt[i] += out[i];
    }
    free(qkv);
    free(att);
}

static void embed(const orc_cfg *c, const orc_weights *w, int64_t n, const int32_t *ids, double *x)
{
    for (int64_t t = 0; t < n; ++t)
        for (int i = 0; i < c->d_model; ++i) x[t * c->d_model + i] = (double)w->emb[(size_t)ids[t] * c->d_model + i];
}

/* score = LNf(x) . w_s + b_s */
static double head(const orc_cfg *c, const orc_weights *w, const double *x)
{
    const int d = c->d_model;
    double a[d];
    layer_norm(x, w->lnf_g, w->lnf_b, c->ln_eps, d, a);
    double acc = 0.0;
    for (int i = 0; i < d; ++i) acc += a[i] * (double)w->w_score[i];
    return acc + (w->b_score ? (double)w->b_score[0] : 0.0);
}

/* Full inference: every token of [prefix; short; candidates] through every layer. */
int orc_full(const orc_cfg *c, const orc_weights *w,
             int64_t P, const int32_t *prefix_ids, int64_t S, const int32_t *short_ids,
             int64_t C, const int32_t *cand_ids, double *scores)
{
    const int d = c->d_model;
    const int64_t n = P + S + C;
    double *x = (double *)malloc(sizeof(double) * (size_t)n * d);
    if (!x) return -1;
    embed(c, w, P, prefix_ids, x);
    embed(c, w, S, short_ids, x + P * d);
    embed(c, w, C, cand_ids, x + (P + S) * d);
    for (int l = 0; l < c->n_layers; ++l) block(c, w, l, P, S, n, 0, x, 0, NULL, NULL, NULL, NULL);
    for (int64_t i = 0; i < C; ++i) scores[i] = head(c, w, x + (P + S + i) * d);
    free(x);
    return 0;
}

/* Pre-inference: the prefix alone; K, V are [L, P, d]. */
int orc_preinfer(const orc_cfg *c, const orc_weights *w, int64_t P, const int32_t *prefix_ids,
                 double *K, double *V)
{
    const int d = c->d_model;
    double *x = (double *)malloc(sizeof(double) * (size_t)P * d);
    if (!x) return -1;
    embed(c, w, P, prefix_ids, x);
    for (int l = 0; l < c->n_layers; ++l)
        block(c, w, l, P, 0, P, 0, x, 0, NULL, NULL, K + (size_t)l * P * d, V + (size_t)l * P * d);
    free(x);
    return 0;
}

/* Rank on cache: short-term and candidate tokens against the stored prefix K, V ([L, P, d]). */
int orc_rank_cached(const orc_cfg *c, const orc_weights *w, int64_t P, const double *K, const double *V,
                    int64_t S, const int32_t *short_ids, int64_t C, const int32_t *cand_ids, double *scores)
{
    const int d = c->d_model;
    const int64_t n = S + C;
    double *x = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1) * d);
    if (!x) return -1;
    embed(c, w, S, short_ids, x);
    embed(c, w, C, cand_ids, x + S * d);
    for (int l = 0; l < c->n_layers; ++l)
        block(c, w, l, P, S, n, P, x, P, K + (size_t)l * P * d, V + (size_t)l * P * d, NULL, NULL);
    for (int64_t i = 0; i < C; ++i) scores[i] = head(c, w, x + (S + i) * d);
    free(x);
    return 0;
}

/* Footprint of psi: K and V rows for every layer (Table 1: 2K x 8 x fp32 x 256 -> 32 MB). */
int64_t orc_kv_bytes(int64_t prefix_len, int64_t n_layers, int64_t d_model, int64_t elem_bytes)
{
    return prefix_len * n_layers * 2 * d_model * elem_bytes;
}

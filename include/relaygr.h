/*
 * relaygr.h - C ABI of the relay-race GR inference hot path (single GPU, sm_100a).
 *
 * The model f is a stack of pre-LayerNorm transformer blocks (softmax
 * multi-head attention, SiLU feed-forward), a final LayerNorm and a linear
 * head producing one logit per candidate item.  A user's sequence is
 * [long-term prefix (P) ; short-term tokens (S) ; candidate items (C)].
 * Attention mask: prefix and short-term tokens are causal over everything
 * before them; a candidate sees the whole prefix, all short-term tokens and
 * itself, never another candidate (the prefix is item-independent, paper
 * Section 3.1).
 *
 * Relay-race inference (paper Section 2.3):
 *     psi <- f([U, S_l, {}, {}], {})                 relaygr_preinfer
 *     f([{}, {}, S~_l, I], psi)                      relaygr_rank
 *     f([U, S_l, S~_l, I], {})                       relaygr_rank_full  (baseline / miss fallback)
 * psi is the per-layer K/V of the prefix (Section 4.1 "Cache semantics"), kept
 * in an HBM-resident paged pool keyed by user id (Section 3.2 "Concurrency
 * inside a special instance", Section 3.3 "HBM as a lifecycle window"), with a
 * pinned-host DRAM tier behind it (Section 3.4).
 *
 * General rules
 *   - Every function returns a relaygr_status (0 = OK, negative = error) and
 *     never throws or aborts.  relaygr_last_error() gives a thread-local text
 *     for the last failing call of the calling thread.
 *   - The CALLER owns all device and pinned-host memory (weights, embedding
 *     table, pool slab, host slab, workspace, inputs, outputs).  The library
 *     owns host-side metadata, a few CUDA events and one small pinned staging
 *     buffer only.  Borrowed pointers must outlive the object that holds them.
 *   - Compute calls are asynchronous on the caller's stream and never
 *     synchronise the device.  Argument errors are returned synchronously and
 *     enqueue nothing.
 *   - "dev" = device pointer, "host" = host pointer.  Streams and events are
 *     passed as void* (cudaStream_t / cudaEvent_t); NULL stream = default.
 *   - A ctx (and a pool) must not be used from two host threads at once.
 *     Calls on one ctx share its workspace: calls on different streams must
 *     be ordered by the caller.
 *   - Model slots (Section 3.2, "Concurrency inside a special instance"): several
 *     ctx created with the same shape and the same weight pointers, each with its
 *     own workspace, may use ONE pool, e.g. pre-infer of some users on one stream
 *     while another ctx ranks other users on a second stream.  The pool orders
 *     producers, consumers, spills and reloads of a user's pages across streams
 *     with events; the host calls themselves must still come from one thread at a time.
 */
#ifndef RELAYGR_H_
#define RELAYGR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RELAYGR_OK = 0,
    RELAYGR_E_INVALID = -1,     /* bad argument, shape or state */
    RELAYGR_E_NOSPACE = -2,     /* pool / host tier / workspace too small */
    RELAYGR_E_EXISTS = -3,      /* user already has an entry */
    RELAYGR_E_MISS = -4,        /* user has no usable cache (caller falls back to relaygr_rank_full) */
    RELAYGR_E_BUSY = -5,        /* a transfer for this user is in flight, or too many reloads in flight */
    RELAYGR_E_CUDA = -6,        /* a CUDA runtime call failed */
    RELAYGR_E_UNSUPPORTED = -7  /* model shape not supported by the kernels */
} relaygr_status;

enum { RELAYGR_DTYPE_F32 = 0, RELAYGR_DTYPE_BF16 = 1 };

/* Where a user's psi currently lives (two-level lookup of Section 3.4). */
enum {
    RELAYGR_TIER_MISS = 0,      /* unknown user */
    RELAYGR_TIER_ALLOCATED = 1, /* pages reserved, pre-infer not yet enqueued */
    RELAYGR_TIER_HBM = 2,       /* resident (its producer may still be running on a stream) */
    RELAYGR_TIER_LOADING = 3,   /* DRAM -> HBM reload enqueued, not yet complete */
    RELAYGR_TIER_HOST = 4       /* spilled to the pinned-host tier only */
};

typedef struct relaygr_ctx relaygr_ctx;
typedef struct relaygr_kv_pool relaygr_kv_pool;

/*
 * Model shape.  d_model = n_heads * d_head.  dtype is the storage type of the
 * embedding table, the matrices, the activations and the K/V pages; vectors
 * are always fp32 and accumulation is always fp32.
 *   F32 : any d_model multiple of 4, d_head in {32, 64}        (CUDA-core kernels)
 *   BF16: d_head = 64, d_model and d_ff multiples of 128       (tcgen05 kernels)
 * page_tokens must be 64.
 *
 * attn_kind selects how a query aggregates the keys it may see (the mask is the same):
 *   RELAYGR_ATTN_SOFTMAX    o_t = sum_j softmax_j(q_t.k_j / sqrt(d_head)) v_j - the block the evaluation
 *                           configurations name.
 *   RELAYGR_ATTN_POINTWISE  o_t = (1 / n_t) sum_j SiLU(q_t.k_j / sqrt(d_head)) v_j, n_t = number of keys visible to t:
 *                           the pointwise aggregated attention of HSTU, the model family of the paper's
 *                           evaluation (Section 5.1), without its relative attention bias.  Everything else
 *                           (the mask, the K/V pool, rank on cache == full inference) is unchanged.
 */
#define RELAYGR_ATTN_SOFTMAX   0
#define RELAYGR_ATTN_POINTWISE 1

typedef struct {
    int32_t n_layers, d_model, n_heads, d_head, d_ff;
    int32_t dtype;
    int32_t page_tokens;
    int64_t vocab;
    float ln_eps;
    int32_t attn_kind;   /* RELAYGR_ATTN_*; zero (softmax) when the struct is zero-initialised */
} relaygr_model_cfg;

/*
 * Parameters, all dev pointers, borrowed.  Linear weights are [out, in]
 * row-major (y = x W^T + b), stacked over layers.  Matrices and emb are in
 * cfg.dtype; every vector is fp32.  A linear bias pointer may be NULL (no bias).
 */
typedef struct {
    const void *emb;                                   /* [vocab, d] */
    const float *ln1_g, *ln1_b, *ln2_g, *ln2_b;        /* [L, d] */
    const void *w_qkv; const float *b_qkv;             /* [L, 3d, d], [L, 3d]; rows 0..d-1 = Q, d..2d-1 = K, 2d.. = V */
    const void *w_o;   const float *b_o;               /* [L, d, d],  [L, d] */
    const void *w1;    const float *b1;                /* [L, F, d],  [L, F] */
    const void *w2;    const float *b2;                /* [L, d, F],  [L, d] */
    const float *lnf_g, *lnf_b, *w_score, *b_score;    /* [d], [d], [d], [1] */
} relaygr_weights;

typedef struct {
    int64_t pages_total, pages_free;         /* HBM pool */
    int64_t host_pages_total, host_pages_free;
    int64_t users_hbm, users_loading, users_host, users_allocated;
    int64_t hits_hbm, hits_loading, hits_host, misses;   /* counted by relaygr_kv_lookup and relaygr_rank */
    int64_t reloads, reload_bytes, spills, spill_bytes;  /* transfers enqueued */
} relaygr_pool_stats;

/* ---- context ------------------------------------------------------------------------------- */

/* Validates the shape, records the (borrowed) weight pointers, selects the current CUDA device. */
int32_t relaygr_create(const relaygr_model_cfg *cfg, const relaygr_weights *w, relaygr_ctx **out);
/*
 * A context without a device, for exercising the pool's bookkeeping (state machine,
 * page accounting, single-flight reload, spill / reload byte-exactness) on a machine
 * with no GPU: "HBM" and host slabs are both plain host memory and tier copies are
 * memcpy.  Every compute call on it returns RELAYGR_E_UNSUPPORTED: there is no CPU path.
 */
int32_t relaygr_create_host_only(const relaygr_model_cfg *cfg, relaygr_ctx **out);
int32_t relaygr_destroy(relaygr_ctx *ctx);
const char *relaygr_last_error(void);

/*
 * Scratch memory for one call: activations for max_rows token rows (sum over the
 * batch of P for pre-infer, S+C for rank, P+S+C for rank_full), metadata for
 * max_users users and max_pages page-table entries, and split-KV partials.
 * relaygr_set_workspace lends the ctx a dev buffer (256-byte aligned) of at
 * least that size; compute calls that need more return RELAYGR_E_NOSPACE.
 */
int32_t relaygr_workspace_bytes(const relaygr_ctx *ctx, int64_t max_rows, int64_t max_users, int64_t max_pages,
                                size_t *out_bytes);
int32_t relaygr_set_workspace(relaygr_ctx *ctx, void *dev, size_t bytes);

/*
 * Kernels never trap, and their internal waits are bounded: a kernel that meets an
 * impossible state records a code in a status word at the start of the workspace - a
 * wait that ran out (RELAYGR_DEVSTATUS_WAIT_TIMEOUT), a token id outside [0, vocab)
 * (RELAYGR_DEVSTATUS_BAD_INDEX; a row that exists is read instead, so no access leaves
 * the table).  The first code stays.  While the word is non-zero the tensor-core
 * kernels of later calls return at once (results undefined, K/V pages not written), so
 * an error cannot pile up.  This call SYNCHRONISES `stream`, then copies the word to
 * *out (0 = healthy).  relaygr_set_workspace clears the word (synchronously).
 */
#define RELAYGR_DEVSTATUS_WAIT_TIMEOUT 1
#define RELAYGR_DEVSTATUS_BAD_INDEX    2
int32_t relaygr_device_status(relaygr_ctx *ctx, void *stream, int32_t *out);

/*
 * Introspection, host only (no GPU, no ctx): the tensor-core attention work list that a
 * bf16 call over users with the given lengths would launch on a GPU with `n_sms` SMs.
 * mode 0 = pre-infer (queries: the prefix, causal), 1 = rank on cache (queries: short-term
 * and candidate tokens; keys: the cached prefix, then the short-term tokens), 2 = full
 * inference (queries: all tokens).  Lengths are host arrays [n_users]; short_len / cand_len
 * are ignored for mode 0.  An item is one 128-row query tile of one head of one user
 * against key blocks [blk0, blk1) of 64 keys; items run in list order, two per SM at a
 * time.  A tile whose key range is split writes partial results that a merge combines.
 *   items  [cap_items][8]  int32: user, head, q0, n_q, blk0, blk1, partial_slot (-1: none),
 *                                  with_self (1: this item folds the candidates' own keys in)
 *   merges [cap_merges][6] int32: user, head, q0, n_q, slot0, n_splits
 * *n_items / *n_merges receive the counts; RELAYGR_E_NOSPACE if a capacity is too small
 * (counts still set), RELAYGR_E_INVALID on bad arguments.  Used by the tests of the
 * split policy (Section 3.2's ranking stage is latency-critical: a launch should not end in
 * a wave of a few long items).
 */
int32_t relaygr_attention_plan(int32_t mode, int32_t n_users, const int32_t *prefix_len,
                               const int32_t *short_len, const int32_t *cand_len,
                               int32_t n_heads, int32_t n_sms,
                               int32_t *items, int32_t cap_items, int32_t *n_items,
                               int32_t *merges, int32_t cap_merges, int32_t *n_merges);

/* ---- paged prefix-KV pool (Section 3.3 sliding window, Section 3.4 DRAM tier) ---------------- */

/*
 * Bytes of one page: [n_layers][K|V][page_tokens][d_model] elements of cfg.dtype,
 * contiguous, so that a page is one copy between tiers.
 */
int32_t relaygr_kv_page_bytes(const relaygr_ctx *ctx, size_t *out_bytes);

/*
 * hbm_slab (dev, 1024-byte aligned) is cut into floor(hbm_bytes / page_bytes)
 * pages; host_slab (pinned host, may be NULL / 0 = no DRAM tier) likewise.
 * The pool never allocates device memory.
 */
int32_t relaygr_kv_pool_create(relaygr_ctx *ctx, void *hbm_slab, size_t hbm_bytes,
                               void *host_slab, size_t host_bytes, relaygr_kv_pool **out);
int32_t relaygr_kv_pool_destroy(relaygr_kv_pool *pool);

/* At most n reloads may be in flight at once (Section 3.4: bounded concurrency); default 8. */
int32_t relaygr_kv_set_max_inflight_reloads(relaygr_kv_pool *pool, int32_t n);

/*
 * Reserve ceil(prefix_len / page_tokens) pages for a new user (state ALLOCATED).
 * page_ids (host, may be NULL) lets the caller pick the pages (they must be
 * free); with NULL the pool picks.  E_EXISTS if the user has an entry in any
 * tier, E_NOSPACE if not enough free pages (the caller evicts: the sliding
 * window policy lives with the caller), E_INVALID if prefix_len < 1.
 */
int32_t relaygr_kv_alloc(relaygr_kv_pool *pool, uint64_t user, int32_t prefix_len, const int32_t *page_ids);

/*
 * Declare an ALLOCATED user's pages filled by the caller (a psi produced elsewhere
 * and copied into the pages returned by relaygr_kv_pages, by work already enqueued
 * on `stream`): the entry becomes HBM-resident, ordered behind that stream's work.
 * E_MISS if unknown, E_INVALID if not ALLOCATED.
 * The pages may have belonged to another user whose spill copy or last rank is still
 * running: call relaygr_kv_wait_pages(pool, user, stream) BEFORE enqueueing the writes.
 * Slots of the last page past prefix_len are never unmasked, but the attention kernels
 * multiply them by a weight of zero: they must hold finite values (zeros will do).
 */
int32_t relaygr_kv_commit(relaygr_kv_pool *pool, uint64_t user, void *stream);

/*
 * Make `stream` wait until every earlier owner of the user's HBM pages has finished with
 * them (Section 3.3: pages change hands as the window slides; a freed page is handed out
 * at once, behind the events of its earlier owners' copies and kernels).  relaygr_preinfer
 * and relaygr_kv_reload_from_host do this themselves; a caller that writes pages directly
 * (relaygr_kv_commit) must.  Enqueues stream waits only.  E_MISS if unknown.
 */
int32_t relaygr_kv_wait_pages(relaygr_kv_pool *pool, uint64_t user, void *stream);

/* Drop the user's entry in every tier.  E_MISS if unknown, E_BUSY while LOADING. */
int32_t relaygr_kv_free(relaygr_kv_pool *pool, uint64_t user);

/*
 * Release the user's HBM pages.  spill_to_host != 0: first copy them to the host
 * tier on `side` (ordered after the user's last enqueued use) and keep the entry
 * in state HOST; E_NOSPACE if the host tier is full (nothing changes).  If a host
 * copy already exists it is reused and nothing is copied.  spill_to_host == 0:
 * the entry stays only if a host copy exists, else it is dropped.
 * Freed pages are handed out again only behind an event that covers the copy and
 * the last use.  E_MISS if unknown or HOST-only, E_BUSY while LOADING.
 */
int32_t relaygr_kv_evict(relaygr_kv_pool *pool, uint64_t user, int32_t spill_to_host, void *side_stream);

/*
 * DRAM -> HBM reload (Section 3.4), idempotent and single-flight: HBM -> OK,
 * nothing enqueued; LOADING -> OK, the in-flight event; HOST -> reserve pages
 * (E_NOSPACE if none) and enqueue the page copies on `side`, state LOADING;
 * unknown / ALLOCATED -> E_MISS; E_BUSY if max_inflight reloads are pending.
 * ready_event_out (may be NULL) receives a cudaEvent_t owned by the pool that
 * completes when the pages are usable (NULL when nothing is pending).  This is
 * also the "pseudo pre-infer" probe of Section 3.4: call it before every rank.
 */
int32_t relaygr_kv_reload_from_host(relaygr_kv_pool *pool, uint64_t user, void *side_stream, void **ready_event_out);

/* Two-level lookup.  tier and prefix_len may be NULL.  Always RELAYGR_OK; a miss is tier == RELAYGR_TIER_MISS. */
int32_t relaygr_kv_lookup(relaygr_kv_pool *pool, uint64_t user, int32_t *tier, int32_t *prefix_len);
/* Copy the user's HBM page ids (host out, capacity cap entries); n_out receives the count. */
int32_t relaygr_kv_pages(relaygr_kv_pool *pool, uint64_t user, int32_t *page_ids_out, int32_t cap, int32_t *n_out);
int32_t relaygr_kv_stats(relaygr_kv_pool *pool, relaygr_pool_stats *out);

/*
 * Test control of a host-only pool (relaygr_create_host_only), so that the states of Section 3.4
 * that need time on a GPU - a reload in flight, pages waiting for a spill copy, the bound on
 * concurrent reloads, a failed transfer - can be held and checked without one.
 *   MANUAL_EVENTS   arg != 0: events recorded from now on stay pending until completed below
 *   COMPLETE_EVENTS complete the arg oldest pending events (arg < 0: all); *out = how many
 *   FAIL_COPIES     the next arg tier copies fail (as a failed cudaMemcpyAsync would)
 *   STREAM_WAITS    *out = number of "stream waits for event" requests the pool has made
 *   PENDING_EVENTS  *out = number of pending events
 * out may be NULL.  E_UNSUPPORTED on a pool that lives on a GPU, E_INVALID for an unknown request.
 */
enum {
    RELAYGR_HOSTCTL_MANUAL_EVENTS = 0,
    RELAYGR_HOSTCTL_COMPLETE_EVENTS = 1,
    RELAYGR_HOSTCTL_FAIL_COPIES = 2,
    RELAYGR_HOSTCTL_STREAM_WAITS = 3,
    RELAYGR_HOSTCTL_PENDING_EVENTS = 4
};
int32_t relaygr_kv_host_backend_control(relaygr_kv_pool *pool, int32_t what, int64_t arg, int64_t *out);

/* ---- the hot path -------------------------------------------------------------------------- */

/*
 * The embedding gather alone (the first step of both passes): out[i, :] = emb[ids[i], :]
 * for n ids, a bit-exact row copy in cfg.dtype.  ids dev int32 [n], out dev [n, d].
 * An id outside [0, vocab) is recorded as RELAYGR_DEVSTATUS_BAD_INDEX in the status word
 * of the lent workspace (if one is lent).
 */
int32_t relaygr_gather(relaygr_ctx *ctx, const int32_t *ids, int64_t n, void *out, void *stream);

/*
 * Pre-inference (Section 2.3, 3.2): run each user's prefix through every layer
 * and write its per-layer K/V rows into the user's pages.  users host [n_users];
 * prefix_ids dev int32, jagged by prefix_off (host int32 [n_users + 1]).  Every
 * user must be ALLOCATED with prefix_len == prefix_off[i+1] - prefix_off[i],
 * else E_INVALID (E_MISS if unknown) and nothing is enqueued.  On success the
 * users become HBM-resident, ordered behind this stream's work.
 */
int32_t relaygr_preinfer(relaygr_ctx *ctx, relaygr_kv_pool *pool, int32_t n_users, const uint64_t *users,
                         const int32_t *prefix_ids, const int32_t *prefix_off, void *stream);

/*
 * Rank on cache (Section 2.3, 3.2): each user's short-term tokens and candidates
 * attend to the cached prefix.  short_ids / cand_ids dev int32, jagged by
 * short_off / cand_off (host int32 [n_users + 1]); S_u = 0 and C_u = 0 are
 * allowed.  scores dev fp32 [cand_off[n_users]], in candidate order.
 * per_user_status (host int32 [n_users], may be NULL) receives each user's
 * RELAYGR_TIER_*.  If any user is not HBM / LOADING the call returns E_MISS and
 * enqueues nothing (Section 3.3: never block on a miss).  For LOADING users
 * the stream waits on the reload event.
 */
int32_t relaygr_rank(relaygr_ctx *ctx, relaygr_kv_pool *pool, int32_t n_users, const uint64_t *users,
                     const int32_t *short_ids, const int32_t *short_off,
                     const int32_t *cand_ids, const int32_t *cand_off,
                     float *scores, int32_t *per_user_status, void *stream);

/* Full inference without cache: the production baseline and the miss fallback (Section 3.3). */
int32_t relaygr_rank_full(relaygr_ctx *ctx, int32_t n_users,
                          const int32_t *prefix_ids, const int32_t *prefix_off,
                          const int32_t *short_ids, const int32_t *short_off,
                          const int32_t *cand_ids, const int32_t *cand_off,
                          float *scores, void *stream);

/*
 * Full inference for callers that cannot hand the library any scratch memory.  (The paper has
 * no counterpart: this is a convenience of this library, not a step of the method.)
 *
 * Who needs it: code that runs where device allocation is off limits and that holds no
 * workspace to lend - a serving process whose whole HBM was carved up at start-up and whose
 * allocator is sealed afterwards, a plug-in running inside another framework's memory pool,
 * a request handler on a latency-critical thread where cudaMalloc's implicit device
 * synchronisation is not acceptable.  For them the miss fallback (relaygr_rank_full) would
 * otherwise be unusable, because that call needs a workspace from relaygr_set_workspace.
 *
 * Same arguments, results and errors as relaygr_rank_full, but the scratch (activations,
 * per-call metadata, split-attention partials, status word) lives in one array of
 * RELAYGR_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that loads the
 * library holds that much memory until the process exits, whether or not this call is used.
 * The call allocates nothing on the device or in pinned memory (it calls no cudaMalloc,
 * cudaFree or allocating library routine); any workspace lent with relaygr_set_workspace is
 * neither needed nor touched.
 *
 *   - A batch whose scratch need (relaygr_workspace_bytes for its rows, users and zero pages)
 *     exceeds RELAYGR_STATIC_SCRATCH_BYTES is rejected with RELAYGR_E_NOSPACE and nothing is
 *     enqueued.  As a guide, one user of a 4-layer d_model-256 bf16 model with a few thousand
 *     tokens fits; large batches do not - lend a workspace and use relaygr_rank_full.
 *   - The first call on each device looks the array's device address up and clears its status
 *     word with a blocking memset; make that first call before any stream capture begins.
 *     The ctx's device must be the current device.
 *   - Every call, from every ctx and thread of the process, shares the one array of its
 *     device, and the array keeps the previous call's contents.  What must start clean is
 *     cleared on `stream` at the start of each call; two calls whose kernels may overlap on
 *     the GPU (different streams without an ordering between them) race - order them.
 *   - If kernels of this call record an internal error, the code is also copied into the
 *     status word of the ctx's lent workspace, when there is one, so that
 *     relaygr_device_status reports it.
 */
#define RELAYGR_STATIC_SCRATCH_BYTES (96u << 20)
int32_t relaygr_rank_full_static(relaygr_ctx *ctx, int32_t n_users,
                                 const int32_t *prefix_ids, const int32_t *prefix_off,
                                 const int32_t *short_ids, const int32_t *short_off,
                                 const int32_t *cand_ids, const int32_t *cand_off,
                                 float *scores, void *stream);

/*
 * Per-kernel timing for benchmarks.  While enabled, every launch of a compute call is
 * bracketed by CUDA events on the call's stream (a few microseconds of overhead per
 * launch: do not leave it on for latency measurements).  relaygr_profile_read waits for
 * the recorded events, returns device milliseconds and launch counts per kernel class
 * accumulated since the previous read, and clears them.  "attention" covers the attention
 * kernel and, when a call splits the key range, its merge kernel.
 */
typedef struct {
    double gather_ln_ms, layernorm_ms, gemm_ms, attention_ms, score_ms;
    int64_t gather_ln_launches, layernorm_launches, gemm_launches, attention_launches, score_launches;
} relaygr_profile;
int32_t relaygr_profile_enable(relaygr_ctx *ctx, int32_t on);
int32_t relaygr_profile_read(relaygr_ctx *ctx, relaygr_profile *out);

/*
 * Kernel launches enqueued by this ctx so far (for benchmark bookkeeping).
 */
int32_t relaygr_launch_count(const relaygr_ctx *ctx, int64_t *out);

#ifdef __cplusplus
}
#endif
#endif /* RELAYGR_H_ */

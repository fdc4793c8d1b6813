// C ABI of the relay-race GR inference path: context, workspace, the three forward
// passes (pre-infer, rank on cache, full inference) and the pool entry points.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/relaygr.h"
#include "forward.hpp"
#include "kv_pool.hpp"

using namespace relaygr;

namespace {
thread_local std::string g_err;
int fail(int code, const std::string &msg) { g_err = msg; return code; }
int fail_cuda(const char *what, cudaError_t e) { g_err = std::string(what) + ": " + cudaGetErrorString(e); return RELAYGR_E_CUDA; }

struct CudaBackend : Backend {
    bool is_cuda() const override { return true; }
    int copy_h2d(void *dst, const void *src, size_t bytes, void *stream) override
    { return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, (cudaStream_t)stream) == cudaSuccess ? 0 : -1; }
    int copy_d2h(void *dst, const void *src, size_t bytes, void *stream) override
    { return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, (cudaStream_t)stream) == cudaSuccess ? 0 : -1; }
    void *event_create() override
    { cudaEvent_t ev = nullptr; return cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess ? (void *)ev : nullptr; }
    void event_destroy(void *ev) override { cudaEventDestroy((cudaEvent_t)ev); }
    int event_record(void *ev, void *stream) override { return cudaEventRecord((cudaEvent_t)ev, (cudaStream_t)stream) == cudaSuccess ? 0 : -1; }
    bool event_done(void *ev) override { return cudaEventQuery((cudaEvent_t)ev) != cudaErrorNotReady; }
    int stream_wait(void *stream, void *ev) override { return cudaStreamWaitEvent((cudaStream_t)stream, (cudaEvent_t)ev, 0) == cudaSuccess ? 0 : -1; }
};
}  // namespace

namespace relaygr { Backend *make_cuda_backend() { return new CudaBackend(); } }

struct relaygr_ctx {
    Forward fwd;            // model shape, weights, workspace, kernel orchestration
    bool host_only = false;
};

struct relaygr_kv_pool {
    relaygr_ctx *ctx;
    Backend *be;
    KvPool *pool;
};

static int check_cfg(const relaygr_model_cfg *c)
{
    if (!c) return fail(RELAYGR_E_INVALID, "cfg is NULL");
    if (c->n_layers < 1 || c->d_model < 1 || c->n_heads < 1 || c->d_ff < 1 || c->vocab < 1)
        return fail(RELAYGR_E_INVALID, "model sizes must be positive");
    if (c->n_heads * c->d_head != c->d_model) return fail(RELAYGR_E_INVALID, "d_model must equal n_heads * d_head");
    if (c->page_tokens != 64) return fail(RELAYGR_E_UNSUPPORTED, "page_tokens must be 64");
    if (c->attn_kind != RELAYGR_ATTN_SOFTMAX && c->attn_kind != RELAYGR_ATTN_POINTWISE)
        return fail(RELAYGR_E_INVALID, "attn_kind must be RELAYGR_ATTN_SOFTMAX or RELAYGR_ATTN_POINTWISE");
    if (c->d_model > 1024) return fail(RELAYGR_E_UNSUPPORTED, "d_model above 1024 is not supported");
    if (c->dtype == RELAYGR_DTYPE_F32) {
        if (c->d_model % 4 || c->d_ff % 4) return fail(RELAYGR_E_UNSUPPORTED, "fp32 model: d_model and d_ff must be multiples of 4");
        if (c->d_head != 32 && c->d_head != 64) return fail(RELAYGR_E_UNSUPPORTED, "fp32 model: d_head must be 32 or 64");
    } else if (c->dtype == RELAYGR_DTYPE_BF16) {
        if (c->d_head != 64) return fail(RELAYGR_E_UNSUPPORTED, "bf16 model: d_head must be 64");
        if (c->d_model % 128 || c->d_ff % 128) return fail(RELAYGR_E_UNSUPPORTED, "bf16 model: d_model and d_ff must be multiples of 128");
    } else {
        return fail(RELAYGR_E_INVALID, "unknown dtype");
    }
    return RELAYGR_OK;
}

static int create_common(const relaygr_model_cfg *cfg, const relaygr_weights *w, bool host_only, relaygr_ctx **out)
{
    if (!out) return fail(RELAYGR_E_INVALID, "out is NULL");
    *out = nullptr;
    const int rc = check_cfg(cfg);
    if (rc != RELAYGR_OK) return rc;
    relaygr_ctx *ctx = new (std::nothrow) relaygr_ctx();
    if (!ctx) return fail(RELAYGR_E_NOSPACE, "out of host memory");
    ctx->host_only = host_only;
    ctx->fwd.cfg = *cfg;
    if (!host_only) {
        if (!w || !w->emb || !w->ln1_g || !w->ln1_b || !w->ln2_g || !w->ln2_b || !w->w_qkv || !w->w_o || !w->w1 || !w->w2 ||
            !w->lnf_g || !w->lnf_b || !w->w_score) {
            delete ctx;
            return fail(RELAYGR_E_INVALID, "a required weight pointer is NULL");
        }
        ctx->fwd.w = *w;
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) { delete ctx; return fail_cuda("no CUDA device (this library has no CPU path)", e); }
        const int irc = ctx->fwd.init_device(dev, g_err);
        if (irc != RELAYGR_OK) { delete ctx; return irc; }
    }
    *out = ctx;
    return RELAYGR_OK;
}

extern "C" {

const char *relaygr_last_error(void) { return g_err.c_str(); }

int32_t relaygr_create(const relaygr_model_cfg *cfg, const relaygr_weights *w, relaygr_ctx **out)
{
    return create_common(cfg, w, false, out);
}

int32_t relaygr_create_host_only(const relaygr_model_cfg *cfg, relaygr_ctx **out)
{
    return create_common(cfg, nullptr, true, out);
}

int32_t relaygr_destroy(relaygr_ctx *ctx)
{
    if (!ctx) return fail(RELAYGR_E_INVALID, "ctx is NULL");
    delete ctx;
    return RELAYGR_OK;
}

int32_t relaygr_workspace_bytes(const relaygr_ctx *ctx, int64_t max_rows, int64_t max_users, int64_t max_pages, size_t *out_bytes)
{
    if (!ctx || !out_bytes || max_rows < 0 || max_users < 0 || max_pages < 0) return fail(RELAYGR_E_INVALID, "bad argument");
    *out_bytes = ctx->fwd.layout(max_rows, max_users, max_pages).total;
    return RELAYGR_OK;
}

int32_t relaygr_set_workspace(relaygr_ctx *ctx, void *dev, size_t bytes)
{
    if (!ctx) return fail(RELAYGR_E_INVALID, "ctx is NULL");
    if (((uintptr_t)dev & 255) != 0) return fail(RELAYGR_E_INVALID, "workspace must be 256-byte aligned");
    if (ctx->host_only) return RELAYGR_OK;
    return ctx->fwd.set_workspace(dev, bytes, g_err);
}

int32_t relaygr_device_status(relaygr_ctx *ctx, void *stream, int32_t *out)
{
    if (!ctx || !out) return fail(RELAYGR_E_INVALID, "bad argument");
    *out = 0;
    if (ctx->host_only) return RELAYGR_OK;
    return ctx->fwd.device_status((cudaStream_t)stream, out, g_err);
}

int32_t relaygr_attention_plan(int32_t mode, int32_t n_users, const int32_t *prefix_len, const int32_t *short_len,
                               const int32_t *cand_len, int32_t n_heads, int32_t n_sms, int32_t *items, int32_t cap_items,
                               int32_t *n_items, int32_t *merges, int32_t cap_merges, int32_t *n_merges)
{
    if (mode < 0 || mode > 2 || n_users < 0 || n_heads < 1 || n_sms < 1 || !n_items || !n_merges || cap_items < 0 || cap_merges < 0 ||
        (n_users > 0 && !prefix_len) || (mode != 0 && n_users > 0 && (!short_len || !cand_len)) || (cap_items > 0 && !items) ||
        (cap_merges > 0 && !merges))
        return fail(RELAYGR_E_INVALID, "bad argument");
    // the same descriptors as relaygr_preinfer / relaygr_rank / relaygr_rank_full build (rows and page-table bases do not
    // enter the plan; only lengths and positions do)
    std::vector<SeqDesc> seqs;
    int64_t row = 0;
    for (int i = 0; i < n_users; ++i) {
        const int P = prefix_len[i], S = mode == 0 ? 0 : short_len[i], C = mode == 0 ? 0 : cand_len[i];
        if (P < 0 || S < 0 || C < 0 || row + (int64_t)P + S + C > INT32_MAX) return fail(RELAYGR_E_INVALID, "bad length");
        SeqDesc s{};
        s.q_row0 = (int32_t)row;
        if (mode == 0) { s.n_q = P; s.q_pos0 = 0; s.n_paged = P; s.n_lin = 0; s.lin_pos0 = P; s.causal_end = P; }
        else if (mode == 1) { s.n_q = S + C; s.q_pos0 = P; s.n_paged = P; s.n_lin = S; s.lin_pos0 = P; s.causal_end = P + S; }
        else { s.n_q = P + S + C; s.q_pos0 = 0; s.n_paged = 0; s.n_lin = P + S; s.lin_pos0 = 0; s.causal_end = P + S; }
        s.lin_row0 = s.self_row0 = s.q_row0;
        row += s.n_q;
        seqs.push_back(s);
    }
    std::vector<AttnItem> it;
    std::vector<AttnMerge> mg;
    build_attention_worklist(seqs, n_heads, n_sms, Forward::kMaxSplitTiles, it, mg);
    *n_items = (int32_t)it.size();
    *n_merges = (int32_t)mg.size();
    if ((int64_t)it.size() > cap_items || (int64_t)mg.size() > cap_merges) return fail(RELAYGR_E_NOSPACE, "plan larger than the arrays given");
    static_assert(sizeof(AttnItem) == 8 * sizeof(int32_t) && sizeof(AttnMerge) == 6 * sizeof(int32_t), "layout of the plan arrays");
    if (!it.empty()) std::memcpy(items, it.data(), it.size() * sizeof(AttnItem));
    if (!mg.empty()) std::memcpy(merges, mg.data(), mg.size() * sizeof(AttnMerge));
    return RELAYGR_OK;
}

int32_t relaygr_profile_enable(relaygr_ctx *ctx, int32_t on)
{
    if (!ctx) return fail(RELAYGR_E_INVALID, "ctx is NULL");
    ctx->fwd.profiling = on != 0;
    return RELAYGR_OK;
}

int32_t relaygr_profile_read(relaygr_ctx *ctx, relaygr_profile *out)
{
    if (!ctx || !out) return fail(RELAYGR_E_INVALID, "bad argument");
    std::memset(out, 0, sizeof(*out));
    if (ctx->host_only) return RELAYGR_OK;
    double ms[Forward::KC_COUNT]; int64_t n[Forward::KC_COUNT];
    const int rc = ctx->fwd.profile_read(ms, n, g_err);
    if (rc) return rc;
    out->gather_ln_ms = ms[Forward::KC_GATHER_LN]; out->gather_ln_launches = n[Forward::KC_GATHER_LN];
    out->layernorm_ms = ms[Forward::KC_LAYERNORM]; out->layernorm_launches = n[Forward::KC_LAYERNORM];
    out->gemm_ms = ms[Forward::KC_GEMM]; out->gemm_launches = n[Forward::KC_GEMM];
    out->attention_ms = ms[Forward::KC_ATTENTION]; out->attention_launches = n[Forward::KC_ATTENTION];
    out->score_ms = ms[Forward::KC_SCORE]; out->score_launches = n[Forward::KC_SCORE];
    return RELAYGR_OK;
}

int32_t relaygr_launch_count(const relaygr_ctx *ctx, int64_t *out)
{
    if (!ctx || !out) return fail(RELAYGR_E_INVALID, "bad argument");
    *out = ctx->fwd.launches;
    return RELAYGR_OK;
}

// ---- pool ------------------------------------------------------------------------------------------

int32_t relaygr_kv_page_bytes(const relaygr_ctx *ctx, size_t *out_bytes)
{
    if (!ctx || !out_bytes) return fail(RELAYGR_E_INVALID, "bad argument");
    const relaygr_model_cfg &c = ctx->fwd.cfg;
    *out_bytes = (size_t)c.n_layers * 2 * 64 * (size_t)c.d_model * (c.dtype == RELAYGR_DTYPE_F32 ? 4 : 2);
    return RELAYGR_OK;
}

int32_t relaygr_kv_pool_create(relaygr_ctx *ctx, void *hbm_slab, size_t hbm_bytes, void *host_slab, size_t host_bytes,
                               relaygr_kv_pool **out)
{
    if (!ctx || !out || !hbm_slab) return fail(RELAYGR_E_INVALID, "bad argument");
    if (((uintptr_t)hbm_slab & 1023) != 0) return fail(RELAYGR_E_INVALID, "hbm_slab must be 1024-byte aligned");
    size_t pb = 0;
    relaygr_kv_page_bytes(ctx, &pb);
    if (hbm_bytes < pb) return fail(RELAYGR_E_NOSPACE, "hbm_bytes holds less than one page");
    if (hbm_bytes / pb > (size_t)1 << 24) return fail(RELAYGR_E_UNSUPPORTED, "more than 2^24 pages");
    // the kernels address the slab as rows of d_model elements through one tensor map with 32-bit row coordinates
    if ((hbm_bytes / pb) * (size_t)ctx->fwd.cfg.n_layers * 128 >= ((size_t)1 << 31))
        return fail(RELAYGR_E_UNSUPPORTED, "pool too large: pages * n_layers * 128 must stay below 2^31 (use several pools)");
    relaygr_kv_pool *p = new (std::nothrow) relaygr_kv_pool();
    if (!p) return fail(RELAYGR_E_NOSPACE, "out of host memory");
    p->ctx = ctx;
    p->be = ctx->host_only ? make_host_backend() : make_cuda_backend();
    p->pool = new KvPool(p->be, ctx->fwd.cfg, hbm_slab, hbm_bytes, host_slab, host_slab ? host_bytes : 0);
    *out = p;
    return RELAYGR_OK;
}

int32_t relaygr_kv_pool_destroy(relaygr_kv_pool *pool)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    delete pool->pool;
    delete pool->be;
    delete pool;
    return RELAYGR_OK;
}

int32_t relaygr_kv_set_max_inflight_reloads(relaygr_kv_pool *pool, int32_t n)
{
    if (!pool || n < 1) return fail(RELAYGR_E_INVALID, "bad argument");
    pool->pool->set_max_inflight(n);
    return RELAYGR_OK;
}

int32_t relaygr_kv_alloc(relaygr_kv_pool *pool, uint64_t user, int32_t prefix_len, const int32_t *page_ids)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    std::string err;
    const int rc = pool->pool->alloc(user, prefix_len, page_ids, err);
    return rc ? fail(rc, err) : rc;
}

int32_t relaygr_kv_commit(relaygr_kv_pool *pool, uint64_t user, void *stream)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    KvPool &kp = *pool->pool;
    UserEntry *e = kp.find(user);
    if (!e) return fail(RELAYGR_E_MISS, "kv_commit: unknown user");
    if (kp.tier_of(*e) != RELAYGR_TIER_ALLOCATED) return fail(RELAYGR_E_INVALID, "kv_commit: user is not in state ALLOCATED");
    const int64_t t = kp.new_ticket(stream);
    if (t == -2) return fail(RELAYGR_E_CUDA, "kv_commit: could not record event");
    e->state = UserState::Resident;
    e->ready_ticket = t;
    e->use_tickets.clear();
    return RELAYGR_OK;
}

int32_t relaygr_kv_wait_pages(relaygr_kv_pool *pool, uint64_t user, void *stream)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    std::string err;
    const int rc = pool->pool->wait_pages_of(user, stream, err);
    return rc ? fail(rc, err) : rc;
}

int32_t relaygr_kv_host_backend_control(relaygr_kv_pool *pool, int32_t what, int64_t arg, int64_t *out)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    const int64_t r = pool->be->control(what, arg);
    if (r < 0) return fail((int)r, r == RELAYGR_E_UNSUPPORTED ? "host_backend_control: only pools of a host-only context have a controllable backend"
                                                               : "host_backend_control: unknown request");
    if (out) *out = r;
    return RELAYGR_OK;
}

int32_t relaygr_kv_free(relaygr_kv_pool *pool, uint64_t user)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    std::string err;
    const int rc = pool->pool->free_user(user, err);
    return rc ? fail(rc, err) : rc;
}

int32_t relaygr_kv_evict(relaygr_kv_pool *pool, uint64_t user, int32_t spill_to_host, void *side_stream)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    std::string err;
    const int rc = pool->pool->evict(user, spill_to_host != 0, side_stream, err);
    return rc ? fail(rc, err) : rc;
}

int32_t relaygr_kv_reload_from_host(relaygr_kv_pool *pool, uint64_t user, void *side_stream, void **ready_event_out)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    std::string err;
    const int rc = pool->pool->reload(user, side_stream, ready_event_out, err);
    return rc ? fail(rc, err) : rc;
}

int32_t relaygr_kv_lookup(relaygr_kv_pool *pool, uint64_t user, int32_t *tier, int32_t *prefix_len)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    return pool->pool->lookup(user, tier, prefix_len, true);
}

int32_t relaygr_kv_pages(relaygr_kv_pool *pool, uint64_t user, int32_t *page_ids_out, int32_t cap, int32_t *n_out)
{
    if (!pool) return fail(RELAYGR_E_INVALID, "pool is NULL");
    std::string err;
    const int rc = pool->pool->pages_of(user, page_ids_out, cap, n_out, err);
    return rc ? fail(rc, err) : rc;
}

int32_t relaygr_kv_stats(relaygr_kv_pool *pool, relaygr_pool_stats *out)
{
    if (!pool || !out) return fail(RELAYGR_E_INVALID, "bad argument");
    pool->pool->stats(out);
    return RELAYGR_OK;
}

// ---- hot path --------------------------------------------------------------------------------------

// A pool may serve every ctx of the same model (model slots); what matters is that pages mean the same thing.
static bool same_model(const relaygr_ctx *a, const relaygr_ctx *b)
{
    const relaygr_model_cfg &x = a->fwd.cfg, &y = b->fwd.cfg;
    return a == b || (x.n_layers == y.n_layers && x.d_model == y.d_model && x.n_heads == y.n_heads && x.d_head == y.d_head &&
                      x.d_ff == y.d_ff && x.dtype == y.dtype && x.page_tokens == y.page_tokens && x.vocab == y.vocab && x.attn_kind == y.attn_kind &&
                      a->host_only == b->host_only && a->fwd.w.w_qkv == b->fwd.w.w_qkv && a->fwd.w.emb == b->fwd.w.emb);
}

static int need_device(relaygr_ctx *ctx)
{
    if (!ctx) return fail(RELAYGR_E_INVALID, "ctx is NULL");
    if (ctx->host_only) return fail(RELAYGR_E_UNSUPPORTED, "host-only context: compute needs a CUDA device, there is no CPU path");
    return RELAYGR_OK;
}

static int check_offsets(const int32_t *off, int n, const char *name, bool allow_empty)
{
    if (!off) return fail(RELAYGR_E_INVALID, std::string(name) + " offsets are NULL");
    if (off[0] != 0) return fail(RELAYGR_E_INVALID, std::string(name) + " offsets must start at 0");
    for (int i = 0; i < n; ++i) {
        if (off[i + 1] < off[i]) return fail(RELAYGR_E_INVALID, std::string(name) + " offsets must not decrease");
        if (!allow_empty && off[i + 1] == off[i]) return fail(RELAYGR_E_INVALID, std::string(name) + ": every user needs at least one token");
    }
    return RELAYGR_OK;
}

int32_t relaygr_gather(relaygr_ctx *ctx, const int32_t *ids, int64_t n, void *out, void *stream)
{
    int rc = need_device(ctx);
    if (rc) return rc;
    if (n < 0 || (n > 0 && (!ids || !out))) return fail(RELAYGR_E_INVALID, "bad argument");
    return ctx->fwd.gather(ids, n, out, (cudaStream_t)stream, g_err);
}

int32_t relaygr_preinfer(relaygr_ctx *ctx, relaygr_kv_pool *pool, int32_t n_users, const uint64_t *users,
                         const int32_t *prefix_ids, const int32_t *prefix_off, void *stream)
{
    int rc = need_device(ctx);
    if (rc) return rc;
    if (!pool || !same_model(pool->ctx, ctx)) return fail(RELAYGR_E_INVALID, "pool was created for a different model");
    if (n_users < 0 || (n_users > 0 && (!users || !prefix_ids))) return fail(RELAYGR_E_INVALID, "bad argument");
    if (n_users == 0) return RELAYGR_OK;
    rc = check_offsets(prefix_off, n_users, "prefix", false);
    if (rc) return rc;
    KvPool &kp = *pool->pool;
    CallDesc call;
    call.mode = MODE_PREINFER;
    std::vector<UserEntry *> entries;
    for (int i = 0; i < n_users; ++i) {
        for (int j = 0; j < i; ++j) if (users[j] == users[i]) return fail(RELAYGR_E_INVALID, "preinfer: a user appears twice in the batch");
        UserEntry *e = kp.find(users[i]);
        if (!e) return fail(RELAYGR_E_MISS, "preinfer: user has no pool entry (call relaygr_kv_alloc first)");
        if (kp.tier_of(*e) != RELAYGR_TIER_ALLOCATED) return fail(RELAYGR_E_INVALID, "preinfer: user is not in state ALLOCATED");
        if (e->prefix_len != prefix_off[i + 1] - prefix_off[i]) return fail(RELAYGR_E_INVALID, "preinfer: prefix length differs from the allocation");
        entries.push_back(e);
    }
    for (int i = 0; i < n_users; ++i) {
        SeqDesc s{};
        const int P = entries[i]->prefix_len;
        s.q_row0 = prefix_off[i]; s.n_q = P; s.q_pos0 = 0;
        s.n_paged = P; s.pt_base = (int32_t)call.page_table.size();
        s.lin_row0 = 0; s.n_lin = 0; s.lin_pos0 = P;
        s.causal_end = P;
        s.score_row0 = 0; s.n_score = 0; s.score_out0 = 0;
        s.self_row0 = s.q_row0;
        call.page_table.insert(call.page_table.end(), entries[i]->pages.begin(), entries[i]->pages.end());
        call.seqs.push_back(s);
    }
    call.n_rows = prefix_off[n_users];
    call.seg_ids[0] = prefix_ids; call.seg_off[0] = prefix_off;
    call.pool_slab = kp.slab();
    call.pool_pages = kp.n_pages();
    rc = ctx->fwd.check_capacity(call, g_err);
    if (rc) return rc;
    for (UserEntry *e : entries)
        if (kp.wait_pages_released(stream, e->pages) != 0) return fail(RELAYGR_E_CUDA, "preinfer: could not order behind page release");
    rc = ctx->fwd.run(call, nullptr, (cudaStream_t)stream, g_err);
    if (rc) return rc;
    const int64_t t = kp.new_ticket(stream);
    if (t == -2) return fail(RELAYGR_E_CUDA, "preinfer: could not record completion event");
    for (UserEntry *e : entries) { e->state = UserState::Resident; e->ready_ticket = t; e->use_tickets.clear(); }
    return RELAYGR_OK;
}

int32_t relaygr_rank(relaygr_ctx *ctx, relaygr_kv_pool *pool, int32_t n_users, const uint64_t *users,
                     const int32_t *short_ids, const int32_t *short_off, const int32_t *cand_ids, const int32_t *cand_off,
                     float *scores, int32_t *per_user_status, void *stream)
{
    int rc = need_device(ctx);
    if (rc) return rc;
    if (!pool || !same_model(pool->ctx, ctx)) return fail(RELAYGR_E_INVALID, "pool was created for a different model");
    if (n_users < 0 || (n_users > 0 && !users)) return fail(RELAYGR_E_INVALID, "bad argument");
    if (n_users == 0) return RELAYGR_OK;
    rc = check_offsets(short_off, n_users, "short-term", true);
    if (rc) return rc;
    rc = check_offsets(cand_off, n_users, "candidate", true);
    if (rc) return rc;
    if ((short_off[n_users] > 0 && !short_ids) || (cand_off[n_users] > 0 && (!cand_ids || !scores)))
        return fail(RELAYGR_E_INVALID, "ids / scores pointer is NULL");
    KvPool &kp = *pool->pool;
    std::vector<UserEntry *> entries((size_t)n_users, nullptr);
    bool miss = false;
    for (int i = 0; i < n_users; ++i) {
        UserEntry *e = kp.find(users[i]);
        const int32_t tier = e ? kp.tier_of(*e) : RELAYGR_TIER_MISS;
        kp.count_hit(tier);
        if (per_user_status) per_user_status[i] = tier;
        if (tier != RELAYGR_TIER_HBM && tier != RELAYGR_TIER_LOADING) miss = true;
        entries[(size_t)i] = e;
    }
    if (miss) return fail(RELAYGR_E_MISS, "rank: at least one user has no HBM-resident prefix cache (see per_user_status)");

    CallDesc call;
    call.mode = MODE_RANK;
    if ((int64_t)short_off[n_users] + (int64_t)cand_off[n_users] > 0x7fffffff) return fail(RELAYGR_E_UNSUPPORTED, "more than 2^31 rows in one call");
    int32_t row = 0;
    for (int i = 0; i < n_users; ++i) {
        const int P = entries[(size_t)i]->prefix_len;
        const int S = short_off[i + 1] - short_off[i], C = cand_off[i + 1] - cand_off[i];
        SeqDesc s{};
        s.q_row0 = row; s.n_q = S + C; s.q_pos0 = P;
        s.n_paged = P; s.pt_base = (int32_t)call.page_table.size();
        s.lin_row0 = row; s.n_lin = S; s.lin_pos0 = P;
        s.causal_end = P + S;
        s.score_row0 = row + S; s.n_score = C; s.score_out0 = cand_off[i];
        s.self_row0 = s.q_row0;
        call.page_table.insert(call.page_table.end(), entries[(size_t)i]->pages.begin(), entries[(size_t)i]->pages.end());
        call.seqs.push_back(s);
        row += S + C;
    }
    call.n_rows = row;
    call.seg_ids[0] = short_ids; call.seg_off[0] = short_off;
    call.seg_ids[1] = cand_ids;  call.seg_off[1] = cand_off;
    call.score_off = cand_off;
    call.pool_slab = kp.slab();
    call.pool_pages = kp.n_pages();
    rc = ctx->fwd.check_capacity(call, g_err);
    if (rc) return rc;
    for (UserEntry *e : entries)
        if (kp.wait_ticket(stream, e->ready_ticket) != 0) return fail(RELAYGR_E_CUDA, "rank: could not order behind the cache producer");
    rc = ctx->fwd.run(call, scores, (cudaStream_t)stream, g_err);
    if (rc) return rc;
    const int64_t t = kp.new_ticket(stream);
    if (t == -2) return fail(RELAYGR_E_CUDA, "rank: could not record completion event");
    for (UserEntry *e : entries) kp.add_use(*e, t);      // every reader counts: several ctx may rank one user on different streams
    return RELAYGR_OK;
}

int32_t relaygr_rank_full(relaygr_ctx *ctx, int32_t n_users, const int32_t *prefix_ids, const int32_t *prefix_off,
                          const int32_t *short_ids, const int32_t *short_off, const int32_t *cand_ids, const int32_t *cand_off,
                          float *scores, void *stream)
{
    int rc = need_device(ctx);
    if (rc) return rc;
    if (n_users < 0) return fail(RELAYGR_E_INVALID, "bad argument");
    if (n_users == 0) return RELAYGR_OK;
    rc = check_offsets(prefix_off, n_users, "prefix", false);
    if (rc) return rc;
    rc = check_offsets(short_off, n_users, "short-term", true);
    if (rc) return rc;
    rc = check_offsets(cand_off, n_users, "candidate", true);
    if (rc) return rc;
    if (!prefix_ids || (short_off[n_users] > 0 && !short_ids) || (cand_off[n_users] > 0 && (!cand_ids || !scores)))
        return fail(RELAYGR_E_INVALID, "ids / scores pointer is NULL");
    CallDesc call;
    call.mode = MODE_FULL;
    int64_t row = 0;
    for (int i = 0; i < n_users; ++i) {
        const int P = prefix_off[i + 1] - prefix_off[i];
        const int S = short_off[i + 1] - short_off[i], C = cand_off[i + 1] - cand_off[i];
        if (row + P + S + C > 0x7fffffff) return fail(RELAYGR_E_UNSUPPORTED, "more than 2^31 rows in one call");
        SeqDesc s{};
        s.q_row0 = (int32_t)row; s.n_q = P + S + C; s.q_pos0 = 0;
        s.n_paged = 0; s.pt_base = 0;
        s.lin_row0 = (int32_t)row; s.n_lin = P + S; s.lin_pos0 = 0;
        s.causal_end = P + S;
        s.score_row0 = (int32_t)row + P + S; s.n_score = C; s.score_out0 = cand_off[i];
        s.self_row0 = s.q_row0;
        call.seqs.push_back(s);
        row += P + S + C;
    }
    call.n_rows = row;
    call.seg_ids[0] = prefix_ids; call.seg_off[0] = prefix_off;
    call.seg_ids[1] = short_ids;  call.seg_off[1] = short_off;
    call.seg_ids[2] = cand_ids;   call.seg_off[2] = cand_off;
    call.score_off = cand_off;
    rc = ctx->fwd.check_capacity(call, g_err);
    if (rc) return rc;
    return ctx->fwd.run(call, scores, (cudaStream_t)stream, g_err);
}

// ---- full inference on scratch that is part of the library image ------------------------------------

namespace {
// The scratch of relaygr_rank_full_static.  In host code this name is only a stand-in for the
// symbol: the address kernels may use comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_static_scratch[RELAYGR_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void *g_static_scratch_addr[kMaxDevices] = {};     // device address of the array, looked up once per device
std::mutex g_static_scratch_mu;

// Copies a non-zero status word of the static scratch into the ctx's lent workspace, where
// relaygr_device_status reads it.
__global__ void forward_status_kernel(const int *from, int *to)
{
    const int v = *from;
    if (v != 0) atomicCAS(to, 0, v);
}

// Device address of the array on the current device `dev`; the first call per device also clears the status word.
int static_scratch_address(int dev, void **out)
{
    std::lock_guard<std::mutex> lock(g_static_scratch_mu);
    if (!g_static_scratch_addr[dev]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return fail_cuda("rank_full_static: cudaGetSymbolAddress of the built-in scratch", e);
        if (!p || ((uintptr_t)p & 255) != 0) return fail(RELAYGR_E_CUDA, "rank_full_static: built-in scratch has no usable device address");
        e = cudaMemset(p, 0, 1024);
        if (e != cudaSuccess) return fail_cuda("rank_full_static: clearing the built-in scratch", e);
        g_static_scratch_addr[dev] = p;
    }
    *out = g_static_scratch_addr[dev];
    return RELAYGR_OK;
}
}  // namespace

int32_t relaygr_rank_full_static(relaygr_ctx *ctx, int32_t n_users, const int32_t *prefix_ids, const int32_t *prefix_off,
                                 const int32_t *short_ids, const int32_t *short_off, const int32_t *cand_ids,
                                 const int32_t *cand_off, float *scores, void *stream)
{
    int rc = need_device(ctx);
    if (rc) return rc;
    if (n_users < 0) return fail(RELAYGR_E_INVALID, "bad argument");
    if (n_users == 0) return RELAYGR_OK;
    // the same argument checks as relaygr_rank_full, made here first so that a bad call enqueues nothing at all
    rc = check_offsets(prefix_off, n_users, "prefix", false);
    if (rc) return rc;
    rc = check_offsets(short_off, n_users, "short-term", true);
    if (rc) return rc;
    rc = check_offsets(cand_off, n_users, "candidate", true);
    if (rc) return rc;
    if (!prefix_ids || (short_off[n_users] > 0 && !short_ids) || (cand_off[n_users] > 0 && (!cand_ids || !scores)))
        return fail(RELAYGR_E_INVALID, "ids / scores pointer is NULL");

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda("rank_full_static: cudaGetDevice", e);
    if (dev != ctx->fwd.device) return fail(RELAYGR_E_INVALID, "rank_full_static: the ctx's device must be the current device");
    if (dev < 0 || dev >= kMaxDevices) return fail(RELAYGR_E_UNSUPPORTED, "rank_full_static: device ordinal out of range");

    const int64_t rows = (int64_t)prefix_off[n_users] + short_off[n_users] + cand_off[n_users];
    const size_t need = ctx->fwd.layout(rows, n_users, 0).total;
    if (need > (size_t)RELAYGR_STATIC_SCRATCH_BYTES) {
        char msg[256];
        std::snprintf(msg, sizeof(msg),
                      "rank_full_static: this batch (%lld token rows, %d users) needs %zu bytes of scratch but the built-in array "
                      "holds %zu; lend a workspace and call relaygr_rank_full",
                      (long long)rows, (int)n_users, need, (size_t)RELAYGR_STATIC_SCRATCH_BYTES);
        return fail(RELAYGR_E_NOSPACE, msg);
    }

    void *scratch = nullptr;
    rc = static_scratch_address(dev, &scratch);
    if (rc) return rc;
    // the array keeps the last call's contents: the status word must start at zero, everything else is
    // written before it is read
    e = cudaMemsetAsync(scratch, 0, 1024, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda("rank_full_static: clearing the status word", e);

    // run the ordinary full-inference call with the built-in array standing in for the lent workspace
    char *lent = ctx->fwd.ws;
    const size_t lent_bytes = ctx->fwd.ws_bytes;
    ctx->fwd.ws = (char *)scratch;
    ctx->fwd.ws_bytes = (size_t)RELAYGR_STATIC_SCRATCH_BYTES;
    rc = relaygr_rank_full(ctx, n_users, prefix_ids, prefix_off, short_ids, short_off, cand_ids, cand_off, scores, stream);
    ctx->fwd.ws = lent;
    ctx->fwd.ws_bytes = lent_bytes;
    if (rc != RELAYGR_OK) return rc;

    if (lent && lent_bytes >= 1024) {
        forward_status_kernel<<<1, 1, 0, (cudaStream_t)stream>>>((const int *)scratch, (int *)lent);
        ctx->fwd.launches += 1;
        e = cudaGetLastError();
        if (e != cudaSuccess) return fail_cuda("rank_full_static: status forwarding", e);
    }
    return RELAYGR_OK;
}

}  // extern "C"

#include "forward.hpp"

#include <algorithm>
#include <cstring>

#include "kernels.cuh"
#include "tc_common.cuh"

namespace relaygr {

namespace {
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
std::string cuda_msg(const char *what, cudaError_t e) { return std::string(what) + ": " + cudaGetErrorString(e); }
}  // namespace

cudaEvent_t Forward::prof_begin(cudaStream_t stream)
{
    if (!profiling) return nullptr;
    cudaEvent_t ev = nullptr;
    if (!prof_spare.empty()) { ev = prof_spare.back(); prof_spare.pop_back(); }
    else if (cudaEventCreate(&ev) != cudaSuccess) return nullptr;
    cudaEventRecord(ev, stream);
    return ev;
}

void Forward::prof_end(int cls, cudaEvent_t start, cudaStream_t stream)
{
    if (!start) return;
    cudaEvent_t ev = nullptr;
    if (!prof_spare.empty()) { ev = prof_spare.back(); prof_spare.pop_back(); }
    else if (cudaEventCreate(&ev) != cudaSuccess) { prof_spare.push_back(start); return; }
    cudaEventRecord(ev, stream);
    prof_pending[cls].push_back({start, ev});
}

int Forward::profile_read(double *ms, int64_t *count, std::string &err)
{
    for (int c = 0; c < KC_COUNT; ++c) {
        ms[c] = 0.0; count[c] = 0;
        for (const EvPair &p : prof_pending[c]) {
            cudaError_t e = cudaEventSynchronize(p.b);
            float t = 0.f;
            if (e == cudaSuccess) e = cudaEventElapsedTime(&t, p.a, p.b);
            if (e != cudaSuccess) { err = cuda_msg("profile read", e); return RELAYGR_E_CUDA; }
            ms[c] += t; count[c] += 1;
            prof_spare.push_back(p.a); prof_spare.push_back(p.b);
        }
        prof_pending[c].clear();
    }
    return RELAYGR_OK;
}

Forward::~Forward()
{
    for (int c = 0; c < KC_COUNT; ++c) for (const EvPair &p : prof_pending[c]) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
    for (cudaEvent_t ev : prof_spare) cudaEventDestroy(ev);
    for (int i = 0; i < kSlots; ++i) if (slot_event[i]) cudaEventDestroy(slot_event[i]);
    if (staging) cudaFreeHost(staging);
}

int Forward::init_device(int dev, std::string &err)
{
    device = dev;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) { err = cuda_msg("cudaGetDeviceProperties", e); return RELAYGR_E_CUDA; }
    if (prop.major != 10) { err = "this library is built for sm_100a (B200) only"; return RELAYGR_E_UNSUPPORTED; }
    n_sms = prop.multiProcessorCount;
    e = cudaMallocHost((void **)&staging, kSlots * kSlotBytes);
    if (e != cudaSuccess) { staging = nullptr; err = cuda_msg("cudaMallocHost (metadata staging)", e); return RELAYGR_E_CUDA; }
    for (int i = 0; i < kSlots; ++i) {
        e = cudaEventCreateWithFlags(&slot_event[i], cudaEventDisableTiming);
        if (e != cudaSuccess) { err = cuda_msg("cudaEventCreate", e); return RELAYGR_E_CUDA; }
    }
    if (cfg.dtype == RELAYGR_DTYPE_BF16) {
        const uint64_t d = (uint64_t)cfg.d_model, F = (uint64_t)cfg.d_ff;
        wmaps.resize((size_t)cfg.n_layers);
        for (int l = 0; l < cfg.n_layers; ++l) {
            const __nv_bfloat16 *wq = (const __nv_bfloat16 *)w.w_qkv + (size_t)l * 3 * d * d;
            int rc = make_tmap_2d_bf16(&wmaps[(size_t)l].qkv, wq, 3 * d, d, d, (uint32_t)kGemmWeightBoxRows, 64);
            rc |= make_tmap_2d_bf16(&wmaps[(size_t)l].kv, wq + d * d, 2 * d, d, d, (uint32_t)kGemmWeightBoxRows, 64);
            rc |= make_tmap_2d_bf16(&wmaps[(size_t)l].wq, wq, d, d, d, (uint32_t)kGemmWeightBoxRows, 64);
            rc |= make_tmap_2d_bf16(&wmaps[(size_t)l].wo, (const __nv_bfloat16 *)w.w_o + (size_t)l * d * d, d, d, d, (uint32_t)kGemmWeightBoxRows, 64);
            rc |= make_tmap_2d_bf16(&wmaps[(size_t)l].w1, (const __nv_bfloat16 *)w.w1 + (size_t)l * F * d, F, d, d, (uint32_t)kGemmWeightBoxRows, 64);
            rc |= make_tmap_2d_bf16(&wmaps[(size_t)l].w2, (const __nv_bfloat16 *)w.w2 + (size_t)l * d * F, d, F, F, (uint32_t)kGemmWeightBoxRows, 64);
            if (ffn_fused_supported((int)d, (int)F)) {
                rc |= make_tmap_2d_bf16(&wmaps[(size_t)l].w2_wide, (const __nv_bfloat16 *)w.w2 + (size_t)l * d * F, d, F, F, 256, 64);
                rc |= make_tmap_2d_bf16(&wmaps[(size_t)l].wo_wide, (const __nv_bfloat16 *)w.w_o + (size_t)l * d * d, d, d, d, 256, 64);
            }
            if (rc != 0) { err = "tensor-map encoding of the weights failed (pointers must be 16-byte aligned)"; return RELAYGR_E_CUDA; }
        }
    }
    return RELAYGR_OK;
}

int Forward::set_workspace(void *dev, size_t bytes, std::string &err)
{
    ws = (char *)dev;
    ws_bytes = dev ? bytes : 0;
    if (ws && ws_bytes >= 1024) {
        cudaError_t e = cudaMemset(ws, 0, 1024);      // the status word starts clean
        if (e != cudaSuccess) { err = cuda_msg("cudaMemset (workspace status)", e); return RELAYGR_E_CUDA; }
    }
    return RELAYGR_OK;
}

int Forward::device_status(cudaStream_t stream, int32_t *out, std::string &err)
{
    *out = 0;
    if (!ws) return RELAYGR_OK;
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e == cudaSuccess) e = cudaMemcpy(out, ws, 4, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { err = cuda_msg("device status read", e); return RELAYGR_E_CUDA; }
    return RELAYGR_OK;
}

WorkspaceLayout Forward::layout(int64_t rows, int64_t users, int64_t pages) const
{
    WorkspaceLayout l{};
    const size_t d = (size_t)cfg.d_model, F = (size_t)cfg.d_ff, es = esize();
    const size_t r = (size_t)rows + 128;    // slack so that 128-row tiles may read past the last row
    size_t at = 0;
    auto take = [&](size_t bytes) { const size_t o = at; at = align_up(at + bytes, 1024); return o; };
    l.status = take(1024);
    l.x = take(r * d * 4);
    l.a = take(r * d * es);
    l.q = take(r * d * es);
    l.k = take(r * d * es);
    l.v = take(r * d * es);
    l.att = take(r * d * es);
    l.hid = take(r * F * es);
    l.x_c = take(r * d * 4);          // the candidate rows of x and of LN1(x), moved together (last layer of a rank call)
    l.a_c = take(r * d * es);
    l.partial_bytes = (size_t)kMaxSplitTiles * 128 * (size_t)(cfg.d_head + 4) * 4;      // rows of m, l, two unused, O (see attention_merge_kernel)
    l.partial = take(l.partial_bytes);
    const size_t n_items = (size_t)cfg.n_heads * ((size_t)rows / 128 + (size_t)users + 1) + 2 * (size_t)kMaxSplitTiles;
    // two descriptor arrays and two work lists: all rows, and the candidate rows of the last layer
    l.meta_bytes = 4 * (((size_t)users + 1) * 5 + 2 * (size_t)users * (sizeof(SeqDesc) / 4) + (size_t)pages + 2 * n_items * (sizeof(AttnItem) / 4) + (size_t)cfg.n_layers + 64);
    l.meta = take(l.meta_bytes);
    l.total = at;
    return l;
}

int Forward::check_capacity(const CallDesc &call, std::string &err) const
{
    if (!ws) { err = "no workspace set (relaygr_set_workspace)"; return RELAYGR_E_NOSPACE; }
    const WorkspaceLayout l = layout(call.n_rows, (int64_t)call.seqs.size(), (int64_t)call.page_table.size());
    if (l.total > ws_bytes) { err = "workspace too small for this call (see relaygr_workspace_bytes)"; return RELAYGR_E_NOSPACE; }
    return RELAYGR_OK;
}

int Forward::upload(const std::vector<int32_t> &blob, size_t dst_off, cudaStream_t stream, std::string &err)
{
    const size_t bytes = blob.size() * 4;
    cudaError_t e;
    if (bytes <= kSlotBytes) {
        const int s = next_slot;
        next_slot = (next_slot + 1) % kSlots;
        if (slot_used[s]) {
            e = cudaEventSynchronize(slot_event[s]);       // only waits if kSlots calls are still in flight
            if (e != cudaSuccess) { err = cuda_msg("cudaEventSynchronize", e); return RELAYGR_E_CUDA; }
        }
        char *src = staging + (size_t)s * kSlotBytes;
        std::memcpy(src, blob.data(), bytes);
        e = cudaMemcpyAsync(ws + dst_off, src, bytes, cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaEventRecord(slot_event[s], stream);
        slot_used[s] = true;
    } else {
        e = cudaMemcpyAsync(ws + dst_off, blob.data(), bytes, cudaMemcpyHostToDevice, stream);   // pageable: staged by the runtime
    }
    if (e != cudaSuccess) { err = cuda_msg("metadata upload", e); return RELAYGR_E_CUDA; }
    return RELAYGR_OK;
}

int Forward::gather(const int32_t *ids, int64_t n, void *out, cudaStream_t stream, std::string &err)
{
    cudaError_t e;
    int *status = (ws && ws_bytes >= 1024) ? reinterpret_cast<int *>(ws) : nullptr;      // the status word of the lent workspace, if any
    if (cfg.dtype == RELAYGR_DTYPE_F32)
        e = launch_gather_rows<float>((const float *)w.emb, cfg.vocab, cfg.d_model, ids, n, (float *)out, status, stream, &launches);
    else
        e = launch_gather_rows<__nv_bfloat16>((const __nv_bfloat16 *)w.emb, cfg.vocab, cfg.d_model, ids, n, (__nv_bfloat16 *)out,
                                              status, stream, &launches);
    if (e != cudaSuccess) { err = cuda_msg("gather", e); return RELAYGR_E_CUDA; }
    return RELAYGR_OK;
}

int Forward::run(const CallDesc &call, float *scores, cudaStream_t stream, std::string &err)
{
    if (cfg.dtype == RELAYGR_DTYPE_F32) return run_t<float>(call, scores, stream, err);
    return run_t<__nv_bfloat16>(call, scores, stream, err);
}

template <typename T>
int Forward::run_t(const CallDesc &call, float *scores, cudaStream_t stream, std::string &err)
{
    const int B = (int)call.seqs.size();
    const int64_t R = call.n_rows;
    if (R == 0) return RELAYGR_OK;
    const int d = cfg.d_model, F = cfg.d_ff, L = cfg.n_layers, H = cfg.n_heads;
    const WorkspaceLayout lay = layout(R, B, (int64_t)call.page_table.size());
    constexpr bool kTensor = sizeof(T) == 2;      // bf16 model: GEMMs and attention run on the tensor cores
    const bool preinfer = call.mode == MODE_PREINFER;
    const int64_t n_scores = (!preinfer && call.score_off) ? call.score_off[B] : 0;
    // The last layer of a rank / full-inference call (bf16 model): only the candidates' hidden states are read afterwards, so
    // every other row needs nothing but its K and V there.  The candidate rows are moved together and the layer's query
    // projection, attention, output projection and feed-forward run on those rows alone.
    const bool compact_last = kTensor && !preinfer;

    auto build_items = [&](const std::vector<SeqDesc> &seqs, std::vector<AttnItem> &items, std::vector<AttnMerge> &merges) {
        build_attention_worklist(seqs, H, n_sms, kMaxSplitTiles, items, merges);
    };

    // ---- metadata blob: row_off | seg_off x3 | score_off | SeqDesc[] | page table | attention items [| the same for the last layer]
    std::vector<int32_t> blob;
    auto put = [&](const int32_t *p, size_t n) { const size_t o = blob.size(); blob.insert(blob.end(), p, p + n); return o; };
    std::vector<int32_t> row_off((size_t)B + 1);
    for (int i = 0; i < B; ++i) row_off[(size_t)i] = call.seqs[(size_t)i].q_row0;
    row_off[(size_t)B] = (int32_t)R;
    const size_t o_row = put(row_off.data(), (size_t)B + 1);
    size_t o_seg[3] = {0, 0, 0};
    for (int s = 0; s < 3; ++s) if (call.seg_off[s]) o_seg[s] = put(call.seg_off[s], (size_t)B + 1);
    const size_t o_score = call.score_off ? put(call.score_off, (size_t)B + 1) : 0;
    const size_t o_seq = put(reinterpret_cast<const int32_t *>(call.seqs.data()), (size_t)B * (sizeof(SeqDesc) / 4));
    const size_t o_pt = call.page_table.empty() ? 0 : put(call.page_table.data(), call.page_table.size());
    std::vector<AttnItem> items, items_c;
    std::vector<AttnMerge> merges, merges_c;
    std::vector<SeqDesc> seqs_c;                  // the candidates of each user as rows of their own (last layer)
    size_t o_items = 0, o_merges = 0, o_seq_c = 0, o_items_c = 0, o_merges_c = 0;
    if (kTensor) {
        build_items(call.seqs, items, merges);
        if (!items.empty()) o_items = put(reinterpret_cast<const int32_t *>(items.data()), items.size() * (sizeof(AttnItem) / 4));
        if (!merges.empty()) o_merges = put(reinterpret_cast<const int32_t *>(merges.data()), merges.size() * (sizeof(AttnMerge) / 4));
        if (compact_last && n_scores > 0) {
            seqs_c = call.seqs;
            for (int u = 0; u < B; ++u) {
                SeqDesc &c = seqs_c[(size_t)u];
                c.self_row0 = c.score_row0;           // where the candidates' own K / V rows (and their x, a rows) are
                c.q_row0 = call.score_off[u];         // where their rows are once moved together
                c.n_q = c.n_score;
                c.q_pos0 = c.causal_end;              // every row is a candidate
                c.score_row0 = call.score_off[u];
            }
            o_seq_c = put(reinterpret_cast<const int32_t *>(seqs_c.data()), (size_t)B * (sizeof(SeqDesc) / 4));
            build_items(seqs_c, items_c, merges_c);
            if (!items_c.empty()) o_items_c = put(reinterpret_cast<const int32_t *>(items_c.data()), items_c.size() * (sizeof(AttnItem) / 4));
            if (!merges_c.empty()) o_merges_c = put(reinterpret_cast<const int32_t *>(merges_c.data()), merges_c.size() * (sizeof(AttnMerge) / 4));
        }
    }
    // one item counter per layer's attention launch (the persistent kernel draws its work from it), zeroed by this upload
    const std::vector<int32_t> zeros((size_t)L, 0);
    const size_t o_ctr = kTensor ? put(zeros.data(), zeros.size()) : 0;
    if (blob.size() * 4 > lay.meta_bytes) { err = "internal: metadata larger than its workspace region"; return RELAYGR_E_NOSPACE; }
    int rc = upload(blob, lay.meta, stream, err);
    if (rc) return rc;

    const int32_t *meta = reinterpret_cast<const int32_t *>(ws + lay.meta);
    const int32_t *d_row_off = meta + o_row;
    const SeqDesc *d_seqs = reinterpret_cast<const SeqDesc *>(meta + o_seq);
    RowSource src{};
    for (int s = 0; s < 3; ++s) {
        const bool on = call.seg_off[s] && call.seg_off[s][B] > 0;
        src.ids[s] = on ? call.seg_ids[s] : nullptr;
        src.off[s] = on ? meta + o_seg[s] : nullptr;
    }
    src.row_off = d_row_off;
    src.n_users = B;

    float *x = reinterpret_cast<float *>(ws + lay.x), *x_c = reinterpret_cast<float *>(ws + lay.x_c);
    T *a = reinterpret_cast<T *>(ws + lay.a), *q = reinterpret_cast<T *>(ws + lay.q), *a_c = reinterpret_cast<T *>(ws + lay.a_c);
    T *kl = reinterpret_cast<T *>(ws + lay.k), *vl = reinterpret_cast<T *>(ws + lay.v);
    T *att = reinterpret_cast<T *>(ws + lay.att), *hid = reinterpret_cast<T *>(ws + lay.hid);

    cudaError_t e = cudaSuccess;
    auto ck = [&](const char *what) -> bool { if (e != cudaSuccess) { err = cuda_msg(what, e); return false; } return true; };

    // per-call tensor maps of the activations (bf16 model)
    int *d_status = reinterpret_cast<int *>(ws + lay.status);
    CUtensorMap &tm_a = act.tm_a, &tm_a_c = act.tm_a_c, &tm_att = act.tm_att, &tm_hid = act.tm_hid, &tm_q = act.tm_q, &tm_k = act.tm_k,
                &tm_v = act.tm_v, &tm_pool = act.tm_pool;
    GemmOutMaps &om_qkv = act.om_qkv, &om_hid = act.om_hid, &om_x = act.om_x, &om_x_c = act.om_x_c;
    const int64_t cand_rows = compact_last ? n_scores : 0;
    const bool maps_cached = act.ws == ws && act.rows == R && act.cand_rows == cand_rows && act.slab == call.pool_slab && act.pages == call.pool_pages;
    if (kTensor && !maps_cached) {
        act.ws = nullptr;                         // not valid until every map below is encoded
        int trc = make_tmap_2d_bf16(&tm_a, a, (uint64_t)R, (uint64_t)d, (uint64_t)d, 128, 64);
        trc |= make_tmap_2d_bf16(&tm_att, att, (uint64_t)R, (uint64_t)d, (uint64_t)d, 128, 64);
        trc |= make_tmap_2d_bf16(&tm_hid, hid, (uint64_t)R, (uint64_t)F, (uint64_t)F, 128, 64);
        trc |= make_tmap_2d_bf16(&tm_q, q, (uint64_t)R, (uint64_t)d, (uint64_t)d, 128, 64);
        trc |= make_tmap_2d_bf16(&tm_k, kl, (uint64_t)R, (uint64_t)d, (uint64_t)d, 64, 64);
        trc |= make_tmap_2d_bf16(&tm_v, vl, (uint64_t)R, (uint64_t)d, (uint64_t)d, 64, 64);
        if (call.pool_slab)
            trc |= make_tmap_2d_bf16(&tm_pool, call.pool_slab, (uint64_t)call.pool_pages * L * 2 * 64, (uint64_t)d, (uint64_t)d, 64, 64);
        else
            tm_pool = tm_k;
        // where the GEMM epilogues store (32-row boxes)
        trc |= make_tmap_2d_bf16(&om_qkv.o[0], q, (uint64_t)R, (uint64_t)d, (uint64_t)d, 32, 64);
        trc |= make_tmap_2d_bf16(&om_qkv.o[1], kl, (uint64_t)R, (uint64_t)d, (uint64_t)d, 32, 64);
        trc |= make_tmap_2d_bf16(&om_qkv.o[2], vl, (uint64_t)R, (uint64_t)d, (uint64_t)d, 32, 64);
        trc |= make_tmap_2d_bf16(&om_hid.o[0], hid, (uint64_t)R, (uint64_t)F, (uint64_t)F, 32, 64);
        trc |= make_tmap_2d_f32(&om_x.o[0], x, (uint64_t)R, (uint64_t)d, (uint64_t)d, 32, 32);
        if (call.pool_slab)
            trc |= make_tmap_2d_bf16(&om_qkv.pool, call.pool_slab, (uint64_t)call.pool_pages * L * 2 * 64, (uint64_t)d, (uint64_t)d, 32, 64);
        else
            om_qkv.pool = om_qkv.o[0];
        om_hid.o[1] = om_hid.o[2] = om_hid.pool = om_hid.o[0];
        om_x.o[1] = om_x.o[2] = om_x.pool = om_x.o[0];
        if (compact_last && n_scores > 0) {
            trc |= make_tmap_2d_bf16(&tm_a_c, a_c, (uint64_t)n_scores, (uint64_t)d, (uint64_t)d, 128, 64);
            trc |= make_tmap_2d_f32(&om_x_c.o[0], x_c, (uint64_t)n_scores, (uint64_t)d, (uint64_t)d, 32, 32);
            om_x_c.o[1] = om_x_c.o[2] = om_x_c.pool = om_x_c.o[0];
        }
        if (trc != 0) { err = "tensor-map encoding of the activations failed"; return RELAYGR_E_CUDA; }
        act.ws = ws; act.rows = R; act.cand_rows = cand_rows; act.slab = call.pool_slab; act.pages = call.pool_pages;
    }
    auto gemm = [&](int64_t M, const T *A, const CUtensorMap &tmA, const T *W, const CUtensorMap *tmW, const GemmOutMaps &om, int N, int K,
                    const Epilogue &ep) {
        cudaEvent_t pe = prof_begin(stream);
        cudaError_t r;
        if constexpr (kTensor) r = launch_gemm_tc(tmA, *tmW, om, M, N, K, ep, d_status, stream, &launches);
        else r = launch_gemm_simt<T>(A, W, M, N, K, ep, stream, &launches);
        prof_end(KC_GEMM, pe, stream);
        return r;
    };
    auto layernorm = [&](const float *xin, int64_t M, const float *g, const float *b) {
        cudaEvent_t pe = prof_begin(stream);
        const cudaError_t r = launch_layernorm<T>(xin, d, M, g, b, cfg.ln_eps, a, stream, &launches);
        prof_end(KC_LAYERNORM, pe, stream);
        return r;
    };
    const LayerMaps *lm = nullptr;

    // the rows the part of a layer after the QKV projection runs on: all of them, or (last layer) the candidates alone
    int64_t M = R;
    float *xm = x;
    const GemmOutMaps *om_xm = &om_x;
    const SeqDesc *seqs_m = d_seqs;
    const AttnItem *items_m = reinterpret_cast<const AttnItem *>(meta + o_items);
    const AttnMerge *merges_m = reinterpret_cast<const AttnMerge *>(meta + o_merges);
    int n_items_m = (int)items.size(), n_merges_m = (int)merges.size();
    bool dead_tail = false;                       // a call without candidates: nothing reads the last layer

    for (int l = 0; l < L; ++l) {
        const bool last = l == L - 1;
        if (last && !preinfer && n_scores == 0) { dead_tail = true; break; }
        const float *g1 = w.ln1_g + (size_t)l * d, *b1n = w.ln1_b + (size_t)l * d;
        if (l == 0) {
            cudaEvent_t pe = prof_begin(stream);
            e = launch_gather_ln<T>((const T *)w.emb, cfg.vocab, d, src, R, g1, b1n, cfg.ln_eps, x, a, d_status, stream, &launches);
            prof_end(KC_GATHER_LN, pe, stream);
        } else {
            e = layernorm(x, R, g1, b1n);
        }
        if (!ck("LayerNorm 1")) return RELAYGR_E_CUDA;

        // fused QKV projection over all rows; K and V only in the last pre-infer layer (psi is K/V alone) and in the last
        // layer of a rank call (the queries of the candidates follow below, on their rows alone)
        const bool kv_only = last && (preinfer || compact_last);
        Epilogue ep{};
        ep.mode = EPI_QKV;
        ep.col0 = kv_only ? d : 0;
        ep.bias = w.b_qkv ? w.b_qkv + (size_t)l * 3 * d + ep.col0 : nullptr;
        ep.d_model = d;
        ep.q = q; ep.k_lin = kl; ep.v_lin = vl;
        ep.seqs = d_seqs; ep.row_off = d_row_off; ep.n_users = B;
        PagedKV paged{};
        if (call.pool_slab) {
            paged.slab = call.pool_slab; paged.pt = meta + o_pt; paged.n_layers = L; paged.d_model = d; paged.layer = l;
        }
        if (preinfer) ep.paged = paged;
        const T *Wqkv = (const T *)w.w_qkv + ((size_t)l * 3 * d + ep.col0) * d;
        lm = kTensor ? &wmaps[(size_t)l] : nullptr;
        e = gemm(R, a, tm_a, Wqkv, lm ? (kv_only ? &lm->kv : &lm->qkv) : nullptr, om_qkv, 3 * d - ep.col0, d, ep);
        if (!ck("QKV projection")) return RELAYGR_E_CUDA;
        if (preinfer && last) break;

        if (last && compact_last) {
            // move the candidates' rows of x and of LN1(x) together, then project their queries
            M = n_scores; xm = x_c; om_xm = &om_x_c;
            seqs_m = reinterpret_cast<const SeqDesc *>(meta + o_seq_c);
            items_m = reinterpret_cast<const AttnItem *>(meta + o_items_c);
            merges_m = reinterpret_cast<const AttnMerge *>(meta + o_merges_c);
            n_items_m = (int)items_c.size(); n_merges_m = (int)merges_c.size();
            cudaEvent_t pe = prof_begin(stream);
            e = launch_compact_rows<T>(x, a, seqs_m, B, meta + o_score, n_scores, d, x_c, a_c, stream, &launches);
            prof_end(KC_LAYERNORM, pe, stream);
            if (!ck("candidate rows")) return RELAYGR_E_CUDA;
            Epilogue eq{};
            eq.mode = EPI_QKV;
            eq.col0 = 0;
            eq.bias = w.b_qkv ? w.b_qkv + (size_t)l * 3 * d : nullptr;
            eq.d_model = d;
            eq.q = q; eq.k_lin = kl; eq.v_lin = vl;
            eq.seqs = seqs_m; eq.row_off = meta + o_score; eq.n_users = B;
            e = gemm(M, a_c, tm_a_c, (const T *)w.w_qkv + (size_t)l * 3 * d * d, lm ? &lm->wq : nullptr, om_qkv, d, d, eq);
            if (!ck("query projection")) return RELAYGR_E_CUDA;
        }

        {
            cudaEvent_t pe = prof_begin(stream);
            if constexpr (kTensor)
                e = launch_attention_tc(tm_q, tm_k, tm_v, tm_pool, items_m, n_items_m, merges_m, n_merges_m, seqs_m, meta + o_pt, L,
                                        l, d, cfg.attn_kind, att, reinterpret_cast<float *>(ws + lay.partial),
                                        reinterpret_cast<int *>(ws + lay.meta) + o_ctr + l, n_sms, d_status, stream, &launches);
            else
                e = launch_attention_simt<T>(q, kl, vl, paged, d_seqs, d_row_off, B, R, H, cfg.d_head, cfg.attn_kind, att, stream, &launches);
            prof_end(KC_ATTENTION, pe, stream);
        }
        if (!ck("attention")) return RELAYGR_E_CUDA;

        if (kTensor && ffn_fused_supported((int)d, (int)F)) {
            // output projection + residual, LayerNorm 2, both feed-forward GEMMs, SiLU and the second residual add in one kernel
            cudaEvent_t pe = prof_begin(stream);
            e = launch_ffn_fused(lm->w1, lm->w2_wide, om_xm->o[0], xm, w.ln2_g + (size_t)l * d, w.ln2_b + (size_t)l * d,
                                 w.b1 ? w.b1 + (size_t)l * F : nullptr, w.b2 ? w.b2 + (size_t)l * d : nullptr, &tm_att, &lm->wo_wide,
                                 w.b_o ? w.b_o + (size_t)l * d : nullptr, M, (int)F, cfg.ln_eps, d_status, stream, &launches);
            prof_end(KC_GEMM, pe, stream);
            if (!ck("output projection + feed-forward")) return RELAYGR_E_CUDA;
            continue;
        }
        Epilogue eo{};
        eo.mode = EPI_RESID; eo.bias = w.b_o ? w.b_o + (size_t)l * d : nullptr; eo.resid = xm; eo.out_f32 = xm;
        e = gemm(M, att, tm_att, (const T *)w.w_o + (size_t)l * d * d, lm ? &lm->wo : nullptr, *om_xm, d, d, eo);
        if (!ck("output projection")) return RELAYGR_E_CUDA;

        e = layernorm(xm, M, w.ln2_g + (size_t)l * d, w.ln2_b + (size_t)l * d);
        if (!ck("LayerNorm 2")) return RELAYGR_E_CUDA;

        Epilogue e1{};
        e1.mode = EPI_STORE; e1.silu = 1; e1.bias = w.b1 ? w.b1 + (size_t)l * F : nullptr; e1.out = hid;
        e = gemm(M, a, tm_a, (const T *)w.w1 + (size_t)l * F * d, lm ? &lm->w1 : nullptr, om_hid, F, d, e1);
        if (!ck("FFN 1")) return RELAYGR_E_CUDA;

        Epilogue e2{};
        e2.mode = EPI_RESID; e2.bias = w.b2 ? w.b2 + (size_t)l * d : nullptr; e2.resid = xm; e2.out_f32 = xm;
        e = gemm(M, hid, tm_hid, (const T *)w.w2 + (size_t)l * d * F, lm ? &lm->w2 : nullptr, *om_xm, d, F, e2);
        if (!ck("FFN 2")) return RELAYGR_E_CUDA;
    }

    if (!dead_tail && n_scores > 0) {
        cudaEvent_t pe = prof_begin(stream);
        e = launch_score(xm, d, seqs_m, B, n_scores, meta + o_score, w.lnf_g, w.lnf_b, cfg.ln_eps, w.w_score, w.b_score,
                         scores, stream, &launches);
        prof_end(KC_SCORE, pe, stream);
        if (!ck("scoring head")) return RELAYGR_E_CUDA;
    }
    return RELAYGR_OK;
}

}  // namespace relaygr

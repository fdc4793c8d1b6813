// Launchers of the device kernels.  Every launcher enqueues on `stream`, returns the
// cudaError_t of the launch and adds the number of kernels it launched to *launches.
#pragma once

#include <cuda.h>

#include <atomic>
#include <utility>

#include "internal.cuh"

namespace relaygr {

// Launch with programmatic stream serialisation: the kernel may begin before its predecessor on the stream has
// finished, and must call grid_dependency_wait() before reading or writing what earlier kernels produce.
// cluster_x > 1 launches thread-block clusters of that many CTAs along x (the grid must be a multiple of it).
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, int cluster_x,
                             Args &&...args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cluster_x > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)cluster_x; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Once-per-device set-up of a kernel (opt-in shared memory size, occupancy query).  A function attribute belongs to the
// device it was set on, so the launchers keep one slot per device: 0 = not set up yet, otherwise the value the set-up
// produced.  Two threads that race through the set-up both store the same value.
constexpr int kMaxDeviceSlots = 64;
struct PerDeviceValue {
    std::atomic<int> slot[kMaxDeviceSlots];
    int get(int dev) const { return dev >= 0 && dev < kMaxDeviceSlots ? slot[dev].load(std::memory_order_acquire) : 0; }
    void set(int dev, int v) { if (dev >= 0 && dev < kMaxDeviceSlots) slot[dev].store(v, std::memory_order_release); }
};

// ---- memory-bound steps (CUDA cores, vectorised loads, warp-shuffle reductions) ----------------

// out[i, :] = emb[ids[i], :], a bit-exact row copy.  An id outside [0, vocab) records STATUS_BAD_INDEX in *err (err may
// be nullptr) and row 0 / vocab - 1 is copied instead, so that no access leaves the table.
template <typename T>
cudaError_t launch_gather_rows(const T *emb, int64_t vocab, int d, const int32_t *ids, int64_t n, T *out, int *err,
                               cudaStream_t stream, int64_t *launches);

// x[r, :] = emb[id(r), :] widened to fp32 (the residual stream); a[r, :] = LN(x[r, :]; g, b) in T.
template <typename T>
cudaError_t launch_gather_ln(const T *emb, int64_t vocab, int d, RowSource src, int64_t n_rows,
                             const float *g, const float *b, float eps, float *x, T *a, int *err,
                             cudaStream_t stream, int64_t *launches);

// a[r, :] = LN(x[r, :]; g, b) in T.
template <typename T>
cudaError_t launch_layernorm(const float *x, int d, int64_t n_rows, const float *g, const float *b, float eps, T *a,
                             cudaStream_t stream, int64_t *launches);

// x_c[i, :] = x[row(i), :], a_c[i, :] = a[row(i), :] for the n_total candidate rows of the call in score order, where
// row(i) = seqs[u].self_row0 + (i - score_off[u]) for the user u that candidate i belongs to (seqs: the compact descriptors).
template <typename T>
cudaError_t launch_compact_rows(const float *x, const T *a, const SeqDesc *seqs, int n_users, const int32_t *score_off, int64_t n_total,
                                int d, float *x_c, T *a_c, cudaStream_t stream, int64_t *launches);

// scores[score_out0 + i] = LN(x[score_row0 + i]; g, b) . w + bias for every user's candidate rows.
cudaError_t launch_score(const float *x, int d, const SeqDesc *seqs, int n_users, int64_t n_scores_total,
                         const int32_t *score_off, const float *g, const float *b, float eps,
                         const float *w, const float *bias, float *scores, cudaStream_t stream, int64_t *launches);

// ---- CUDA-core GEMM and attention (the fp32 model) ---------------------------------------------

// C[m, n] = sum_k A[m, k] W[n, k], m < M, n < N, then `epi`.
template <typename T>
cudaError_t launch_gemm_simt(const T *A, const T *W, int64_t M, int N, int K, const Epilogue &epi,
                             cudaStream_t stream, int64_t *launches);

// One warp per (row, head): attention (softmax, or pointwise SiLU for ATTN_POINTWISE) under the SeqDesc mask.  out [n_rows, d] in T.
template <typename T>
cudaError_t launch_attention_simt(const T *q, const T *k_lin, const T *v_lin, PagedKV paged, const SeqDesc *seqs,
                                  const int32_t *row_off, int n_users, int64_t n_rows, int n_heads, int d_head, int attn_kind,
                                  T *out, cudaStream_t stream, int64_t *launches);

// ---- tensor-core kernels (the bf16 model) -------------------------------------------------------------

// The tensor-core GEMM for [M, K] x [N, K]^T (N % 128 == 0) runs on CTA pairs (256 x 256 tiles, tcgen05 cta_group::2)
// when N is a multiple of 256 and the pair's deeper pipeline has enough work to pay for itself: a mainloop of K >= 512,
// or at least four tiles per pair of SMs (measured on the model's shapes).  Otherwise single CTAs with 128 x 128 tiles.
// Either way a CTA loads W in boxes of 128 rows.
inline bool gemm_pair(int64_t M, int N, int K)
{
    return N % 256 == 0 && (K >= 512 || ((M + 255) / 256) * (N / 256) >= 4 * 74);
}
constexpr int kGemmWeightBoxRows = 128;

// Where a GEMM's epilogue stores: tensor maps with a 32-row box of 128 bytes and the 128-byte swizzle.
// EPI_STORE: o[0] = out [M, N] bf16.  EPI_RESID: o[0] = the fp32 residual stream [M, N] (tile added in place).
// EPI_QKV: o[0] = q, o[1] = k_lin, o[2] = v_lin, each [M, d] bf16 (o[1], o[2] are not used when K / V go to pages);
// pool = the pool slab viewed as [pages * L * 2 * 64, d] (used when K / V go to pages, else any valid map).
struct GemmOutMaps { CUtensorMap o[3]; CUtensorMap pool; };

// C[m, n] = sum_k A[m, k] W[n, k] on tcgen05; tmA covers A [M, K] with a 128-row box, tmB covers W [N, K]
// with a box of kGemmWeightBoxRows rows, both 64 columns wide with the 128-byte swizzle.  N % 128 == 0, K % 64 == 0.
// err is a device status word: kernels record a code there instead of hanging or trapping.
cudaError_t launch_gemm_tc(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmOutMaps &om, int64_t M, int N, int K,
                           const Epilogue &epi, int *err, cudaStream_t stream, int64_t *launches);

// The feed-forward half of a block in one kernel, x <- x + W2 SiLU(W1 LN(x; g, b) + b1) + b2, for the shapes
// ffn_fused_supported() accepts (d_model = 256, d_ff a multiple of 128 up to 2048): LayerNorm, both GEMMs, SiLU and the
// residual add without a round trip of the normalised or hidden activations through global memory.  tmW1: W1 [d_ff, 256]
// in boxes of 128 rows x 64 columns; tmW2: W2 [256, d_ff] in boxes of 256 rows x 64 columns; tmX: the fp32 residual stream
// [M, 256] in boxes of 32 rows x 32 columns (read by the LayerNorm of the projection form, target of the add-reduction);
// all with the 128-byte swizzle.
// With tmAtt / tmWo (both or neither) the attention block's output projection runs first in the same kernel:
// mid = x + att Wo^T + bo, x <- mid + W2 SiLU(W1 LN(mid) + b1) + b2.  tmAtt: att [M, 256] bf16 in boxes of 128 rows x 64
// columns; tmWo: Wo [256, 256] in boxes of 256 rows x 64 columns.
bool ffn_fused_supported(int d_model, int d_ff);
cudaError_t launch_ffn_fused(const CUtensorMap &tmW1, const CUtensorMap &tmW2, const CUtensorMap &tmX, const float *x, const float *g,
                             const float *b, const float *b1, const float *b2, const CUtensorMap *tmAtt, const CUtensorMap *tmWo,
                             const float *bo, int64_t M, int d_ff, float eps, int *err, cudaStream_t stream, int64_t *launches);

// Flash-style attention on tcgen05 (d_head = 64) over the work items, then the merge of split items.  attn_kind: ATTN_SOFTMAX, or
// ATTN_POINTWISE (weights SiLU(q.k / sqrt(d_h)) divided by the number of visible keys).
// tmQ: [rows, d] box 128 x 64; tmK / tmV: the call's transient K / V rows, box 64 x 64; tmPool: the pool
// slab viewed as [pages * L * 2 * 64, d], box 64 x 64 (pass tmK when the call has no pool).
// The kernel is persistent: min(n_items, 2 x n_sms) CTAs draw item indices from *next_item, a device counter that must be
// zero when the kernel starts and belongs to this launch alone (the kernel leaves it non-zero).
cudaError_t launch_attention_tc(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV, const CUtensorMap &tmPool,
                                const AttnItem *items, int n_items, const AttnMerge *merges, int n_merges, const SeqDesc *seqs,
                                const int32_t *pt, int n_layers, int layer, int d_model, int attn_kind, __nv_bfloat16 *out,
                                float *partial, int *next_item, int n_sms, int *err, cudaStream_t stream, int64_t *launches);

}  // namespace relaygr

// Structures shared by the host runtime and the kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/relaygr.h"

namespace relaygr {

// One user of a call.  Rows are the token rows the call computes (activations are
// dense [n_rows, d], users back to back).  Keys come from two places: "paged" keys
// (the pool, through the page table) at sequence positions 0 .. n_paged-1, and
// "linear" keys (rows of the call's transient K/V buffers) at positions
// lin_pos0 .. lin_pos0+n_lin-1.  Mask: a query at position t < causal_end sees
// keys at positions <= t; a query at t >= causal_end (a candidate) sees keys at
// positions < causal_end plus its own K/V row, which is row self_row0 + i of the transient K/V buffers for the user's
// query row i (the query rows themselves may sit elsewhere: the last layer of a rank call runs on the candidate rows alone,
// moved together, while their K/V stay where the projection of all rows wrote them).
struct SeqDesc {
    int32_t q_row0, n_q, q_pos0;
    int32_t n_paged, pt_base;
    int32_t lin_row0, n_lin, lin_pos0;
    int32_t causal_end;
    int32_t score_row0, n_score, score_out0;
    int32_t self_row0;
};

// Where the token ids of the rows come from: up to three jagged segments per user, in order.
struct RowSource {
    const int32_t *ids[3];   // device id arrays (nullptr = segment absent)
    const int32_t *off[3];   // device offsets [n_users + 1] of each segment
    const int32_t *row_off;  // device [n_users + 1]
    int32_t n_users;
};

// Addressing of the paged pool: page = [L][K|V][64][d].
struct PagedKV {
    void *slab;
    const int32_t *pt;       // device page table (all users of the call, concatenated)
    int32_t n_layers, d_model, layer;
};

// One unit of tensor-core attention work: a 128-row query tile of one head of one user
// against the key blocks [blk0, blk1) of that user (128 keys each; paged blocks first,
// then linear blocks).  partial_slot >= 0: write (m, l, O) to that slot for a later merge.
struct AttnItem {
    int32_t seq, head, q0, n_q;
    int32_t blk0, blk1;
    int32_t partial_slot;
    int32_t with_self;        // fold the candidate's own key in (exactly one split of a tile does)
};

struct AttnMerge {
    int32_t seq, head, q0, n_q;
    int32_t slot0, n_splits;
};

// Codes a kernel may record in the status word at the start of the workspace (relaygr_device_status; 0 = healthy).
// The first code recorded stays.
enum DeviceStatus : int { STATUS_OK = 0, STATUS_WAIT_TIMEOUT = RELAYGR_DEVSTATUS_WAIT_TIMEOUT, STATUS_BAD_INDEX = RELAYGR_DEVSTATUS_BAD_INDEX };

enum EpiMode : int32_t { EPI_STORE = 0, EPI_RESID = 1, EPI_QKV = 2 };

// How a query aggregates the keys it may see (relaygr_model_cfg.attn_kind).
enum AttnKind : int32_t { ATTN_SOFTMAX = 0, ATTN_POINTWISE = 1 };

// What a GEMM does with its fp32 accumulators: C[m, n] = sum_k A[m,k] W[n,k].
struct Epilogue {
    int32_t mode;
    int32_t silu;                 // EPI_STORE: apply SiLU after the bias
    const float *bias;            // [N] (already offset to this layer), may be nullptr
    void *out;                    // EPI_STORE: [M, N] in the model dtype
    const float *resid;           // EPI_RESID: fp32 [M, N] read ...
    float *out_f32;               // ... and fp32 [M, N] written (may alias resid)
    // EPI_QKV: column c of the full [3d] output goes to q (c < d), K (d <= c < 2d) or V.
    int32_t col0;                 // first output column this GEMM computes (0, or d for K/V only)
    int32_t d_model;
    void *q;                      // [M, d]
    void *k_lin, *v_lin;          // [M, d] transient K/V (used when paged.slab == nullptr)
    PagedKV paged;                // else K/V rows are scattered into pages
    const SeqDesc *seqs;          // per-user descriptors (paged scatter needs row -> user -> page)
    const int32_t *row_off;
    int32_t n_users;
};

// Programmatic dependent launch: a kernel launched with launch_dependent() may start while the kernel before it on
// the stream is still running.  It does its set-up (barriers, TMEM, descriptor prefetch), then calls
// grid_dependency_wait() before it touches anything that earlier kernels wrote; grid_launch_dependents() lets the
// kernel after it start its own set-up as soon as every CTA of this one has begun.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ int find_user(const int32_t *row_off, int n_users, int row)
{
    // largest u with row_off[u] <= row
    int lo = 0, hi = n_users;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (row_off[mid] <= row) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ size_t page_elem_offset(const PagedKV &p, int page, int kv, int slot)
{
    return ((((size_t)page * p.n_layers + p.layer) * 2 + kv) * 64 + slot) * (size_t)p.d_model;
}

template <typename T> struct Num;
template <> struct Num<float> {
    static __device__ __forceinline__ float to_f(float v) { return v; }
    static __device__ __forceinline__ float from_f(float v) { return v; }
};
template <> struct Num<__nv_bfloat16> {
    static __device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
    static __device__ __forceinline__ __nv_bfloat16 from_f(float v) { return __float2bfloat16_rn(v); }
};

}  // namespace relaygr

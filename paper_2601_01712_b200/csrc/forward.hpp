// Orchestration of one forward pass (pre-infer, rank on cache, or full inference):
// builds the per-call metadata, uploads it, and enqueues the kernels layer by layer.
#pragma once

#include <cstdint>
#include <string>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/relaygr.h"
#include "internal.cuh"
#include "kernels.cuh"

namespace relaygr {

enum CallMode { MODE_PREINFER = 0, MODE_RANK = 1, MODE_FULL = 2 };

// The attention work list of one call (host only): items in launch order, and the merges of split items.
void build_attention_worklist(const std::vector<SeqDesc> &seqs, int n_heads, int n_sms, int64_t max_split_tiles,
                              std::vector<AttnItem> &items, std::vector<AttnMerge> &merges);

struct CallDesc {
    int mode = MODE_RANK;
    std::vector<SeqDesc> seqs;
    std::vector<int32_t> page_table;
    int64_t n_rows = 0;
    const int32_t *seg_ids[3] = {nullptr, nullptr, nullptr};   // device
    const int32_t *seg_off[3] = {nullptr, nullptr, nullptr};   // host, [n_users + 1]
    const int32_t *score_off = nullptr;                        // host, [n_users + 1]
    void *pool_slab = nullptr;
    int64_t pool_pages = 0;
};

struct WorkspaceLayout {
    size_t status, x, a, q, k, v, att, hid, x_c, a_c, partial, meta, total;
    size_t meta_bytes, partial_bytes;
};

struct Forward {
    relaygr_model_cfg cfg{};
    relaygr_weights w{};
    char *ws = nullptr;
    size_t ws_bytes = 0;
    int64_t launches = 0;
    int device = 0;
    int n_sms = 148;

    // tensor maps of the weights (bf16 model), one set per layer
    struct LayerMaps { CUtensorMap qkv, kv, wq, wo, w1, w2, w2_wide, wo_wide; };      // *_wide: boxes of 256 rows (fused out-proj + feed-forward)
    std::vector<LayerMaps> wmaps;

    // tensor maps of the activations (bf16 model): a function of the workspace, the row counts and the pool slab alone, so
    // calls of the same shape - the usual case in serving - reuse them instead of encoding some twenty maps per call
    struct ActMaps {
        const char *ws = nullptr; int64_t rows = -1, cand_rows = -1; const void *slab = nullptr; int64_t pages = -1;
        CUtensorMap tm_a, tm_a_c, tm_att, tm_hid, tm_q, tm_k, tm_v, tm_pool;
        GemmOutMaps om_qkv, om_hid, om_x, om_x_c;
    } act;

    // pinned staging ring for the per-call metadata
    static constexpr int kSlots = 4;
    static constexpr size_t kSlotBytes = 2u << 20;
    char *staging = nullptr;
    cudaEvent_t slot_event[kSlots] = {};
    bool slot_used[kSlots] = {};
    int next_slot = 0;

    // optional per-kernel-class timing with CUDA events on the call's stream
    enum KernelClass { KC_GATHER_LN = 0, KC_LAYERNORM, KC_GEMM, KC_ATTENTION, KC_SCORE, KC_COUNT };
    bool profiling = false;
    struct EvPair { cudaEvent_t a, b; };
    std::vector<EvPair> prof_pending[KC_COUNT];
    std::vector<cudaEvent_t> prof_spare;
    cudaEvent_t prof_begin(cudaStream_t stream);
    void prof_end(int cls, cudaEvent_t start, cudaStream_t stream);
    int profile_read(double *ms, int64_t *count, std::string &err);

    ~Forward();
    int init_device(int dev, std::string &err);
    WorkspaceLayout layout(int64_t rows, int64_t users, int64_t pages) const;
    int check_capacity(const CallDesc &call, std::string &err) const;
    int run(const CallDesc &call, float *scores, cudaStream_t stream, std::string &err);
    int gather(const int32_t *ids, int64_t n, void *out, cudaStream_t stream, std::string &err);
    int set_workspace(void *dev, size_t bytes, std::string &err);
    int device_status(cudaStream_t stream, int32_t *out, std::string &err);

    size_t esize() const { return cfg.dtype == RELAYGR_DTYPE_F32 ? 4 : 2; }
    static constexpr int64_t kMaxSplitTiles = 1536;   // capacity of the split-KV partial buffer, in 128-row tiles

private:
    template <typename T> int run_t(const CallDesc &call, float *scores, cudaStream_t stream, std::string &err);
    int upload(const std::vector<int32_t> &blob, size_t dst_off, cudaStream_t stream, std::string &err);
};

}  // namespace relaygr

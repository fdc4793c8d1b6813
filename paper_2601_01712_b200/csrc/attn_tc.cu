// Flash-style attention on tcgen05 for the bf16 model (d_head = 64), serving all three passes:
// pre-infer (causal over the user's own pages), rank on cache (prefix pages through the page
// table + short-term rows + the candidate's own row) and full inference (linear K/V rows).
//
// A work item = a 128-row query tile of one head of one user against a range of that user's
// 64-key blocks (one block = one 64-token page of the pool, or 64 rows of the call's transient
// K/V buffers; one 8 KB TMA box each for K and V).  Per block:
//     S = Q K^T   tcgen05.mma M=128 N=64 K=64, operands in shared memory, S in TMEM
//     softmax     128 threads, one row each: S row -> registers, running max, p = 2^(s c - m c),
//                 bf16 P written back to TMEM
//     O += P V    tcgen05.mma M=128 N=64 K=64, A = P from TMEM, B = V in shared memory (MN-major),
//                 O accumulated in TMEM
// S and P are double-buffered in TMEM, so the MMA warp runs one block ahead of the softmax and
// the tensor pipe never waits for it in steady state.  The exponentials of a block are taken
// against the running maximum as it stood before the block; only when the block's row sum shows
// that some exponent may have exceeded 2^8 is the block maximum computed, the running maximum
// raised, O rescaled in TMEM (after the pending PV has drained) and the block redone - so no
// maximum is on the fast path, every exponent that is kept stays below 2^8, and rescales are rare.
// A candidate's own key (it sees the prefix, the short-term tokens and itself) is one more block
// of the same pipeline: the 64-row group of the call's K / V that holds the candidate's row, with
// a diagonal mask (own_key_blocks).
//
// The kernel is persistent: two CTAs per SM, each drawing items from a counter until the list is
// exhausted.  The TMA producer and the MMA issuer run on into the next item (its Q, its first K / V
// tiles, its first two S) while the softmax warps finish the current one, so launch, set-up and
// load latencies are paid once per CTA instead of once per item; barrier phases and pipeline
// stages are counted over the CTA's running block index.
//
// Warp roles (192 threads): warp 0 = TMA producer (and the item counter), warp 1 = TMEM owner +
// MMA issuer, warps 2-5 = softmax / correction / epilogue (TMEM lane quadrant = warp index % 4).
#include <algorithm>

#include "kernels.cuh"
#include "tc_common.cuh"

namespace relaygr {

namespace {

constexpr int kQTile = 128, kKeys = 64, kDh = 64;
constexpr int kQBytes = kQTile * kDh * 2;           // 16 KB
constexpr int kKVBytes = kKeys * kDh * 2;           // 8 KB per K or V tile
#ifndef RELAYGR_ATTN_OFFLOAD
#define RELAYGR_ATTN_OFFLOAD 1
#endif
constexpr bool kOffload = RELAYGR_ATTN_OFFLOAD != 0;                       // a quarter of the exponentials runs on the FMA pipe (exp2_fma_pipe)
constexpr int kStagesKV = 4;
constexpr int kSmemBytes = kQBytes + 2 * kStagesKV * kKVBytes + 1024 + 512;
constexpr uint32_t kTmemCols = 256;                 // S[2]: 0..127, P[2]: 128..191, O: 192..255
constexpr uint32_t kColS = 0, kColP = 128, kColO = 192;
constexpr int kPartStride = kDh + 4;                // floats per row of a split partial: m, l, two unused, then O (16-byte aligned rows)
constexpr float kRowSumLimit = 256.f;               // a block's row sum above this: some p may exceed 2^8 -> redo against a raised maximum

struct Bars {
    uint64_t q_full, q_empty;
    uint64_t k_full[kStagesKV], k_empty[kStagesKV], v_full[kStagesKV], v_empty[kStagesKV];
    uint64_t s_full[2], p_full[2], p_free[2];
    uint64_t item_full[2], item_empty[2];
    int ring[2];                 // item indices on their way from the producer to the other warps (-1: no more)
    uint32_t tmem_slot;
    int abort_flag;
};

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Packed pairs of fp32 (sm_100 executes fma / add on two lanes of a 64-bit register per instruction).
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// 2^x for a packed pair WITHOUT the XU pipe: x is rounded to the nearest integer n by adding 1.5 * 2^23 (n then sits in
// the low mantissa bits), a cubic gives 2^(x - n) on [-0.5, 0.5] (relative error 7.5e-5, far below the bf16 rounding of P
// that follows) and n is added to the exponent field as an integer.  x is clamped to [-126, 126] first: below that the
// result is ~1e-38 instead of 0 (a masked key's -inf included: its weight stays negligible), above it the row-sum check
// of the caller fails and the block is redone against a true maximum.
__device__ __forceinline__ void exp2_fma_pipe(uint64_t x2, float &p0, float &p1)
{
    float x0, x1;
    unpack2(x2, x0, x1);
    x0 = fminf(fmaxf(x0, -126.f), 126.f);
    x1 = fminf(fmaxf(x1, -126.f), 126.f);
    const uint64_t xc = pack2(x0, x1);
    const uint64_t r2 = add2(xc, pack2(12582912.f, 12582912.f));
    const uint64_t n2 = add2(r2, pack2(-12582912.f, -12582912.f));
    const uint64_t f2 = fma2(n2, pack2(-1.f, -1.f), xc);
    uint64_t q2 = fma2(pack2(0.0551716685f, 0.0551716685f), f2, pack2(0.2426111251f, 0.2426111251f));
    q2 = fma2(q2, f2, pack2(0.6932609677f, 0.6932609677f));
    q2 = fma2(q2, f2, pack2(0.9999280572f, 0.9999280572f));
    float r0, r1, q0, q1;
    unpack2(r2, r0, r1);
    unpack2(q2, q0, q1);
    p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(r0) << 23));
    p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(r1) << 23));
}

// x if a == b, else y - as a select, never a branch (a per-lane `b` compared against every unrolled `a` otherwise
// compiles to a jump table that diverges 32 ways)
__device__ __forceinline__ uint32_t select_eq(int a, int b, uint32_t x, uint32_t y)
{
    uint32_t r;
    asm("{\n .reg .pred p;\n setp.eq.s32 p, %1, %2;\n selp.b32 %0, %3, %4, p;\n}\n" : "=r"(r) : "r"(a), "r"(b), "r"(x), "r"(y));
    return r;
}

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// The candidates' own keys.  A candidate sees the prefix, the short-term tokens and itself: its own K / V row is not among
// the key blocks above, so every 64-row group of the tile that holds a candidate row is appended to the item as one more
// key block - rows self_row0 + q0 + 64 t .. + 63 of the call's K / V - with a diagonal mask: row r sees key r alone.
// d0 = the first such group, n_diag = how many (0 when the item has no candidates, or is not the split that owns them).
__device__ __forceinline__ void own_key_blocks(const AttnItem &it, const SeqDesc &sd, int &d0, int &n_diag)
{
    const int first_cand = max(0, sd.causal_end - (sd.q_pos0 + it.q0));      // first candidate row of the tile
    d0 = 0;
    n_diag = 0;
    if (it.with_self && first_cand < it.n_q) {
        d0 = first_cand / kKeys;
        n_diag = (it.n_q + kKeys - 1) / kKeys - d0;
    }
}

// kPointwise: pointwise aggregated attention (HSTU style) - the weight of a visible key is SiLU(q.k / sqrt(d_h)) and the
// sum is divided by the number of visible keys; no running maximum, no row sum, no rescaling of O.
template <bool kPointwise>
__global__ void __launch_bounds__(192, 2)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKlin,
                    const __grid_constant__ CUtensorMap tmVlin, const __grid_constant__ CUtensorMap tmPool,
                    const AttnItem *__restrict__ items, int n_items, int *__restrict__ next_item, const SeqDesc *__restrict__ seqs,
                    const int32_t *__restrict__ pt, int n_layers, int layer, int d_model, __nv_bfloat16 *__restrict__ out,
                    float *__restrict__ partial, int *err)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = smem;
    uint8_t *sK = smem + kQBytes;
    uint8_t *sV = sK + kStagesKV * kKVBytes;
    Bars *bars = reinterpret_cast<Bars *>(sV + kStagesKV * kKVBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // set-up that touches nothing earlier kernels wrote; it may run while the previous kernel is still finishing
    if (threadIdx.x == 0) {
        tc::mbar_init(&bars->q_full, 1); tc::mbar_init(&bars->q_empty, 1);
        for (int s = 0; s < kStagesKV; ++s) {
            tc::mbar_init(&bars->k_full[s], 1); tc::mbar_init(&bars->k_empty[s], 1);
            tc::mbar_init(&bars->v_full[s], 1); tc::mbar_init(&bars->v_empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            tc::mbar_init(&bars->s_full[b], 1);
            tc::mbar_init(&bars->p_full[b], 128); tc::mbar_init(&bars->p_free[b], 1);
            tc::mbar_init(&bars->item_full[b], 1); tc::mbar_init(&bars->item_empty[b], 5);     // MMA warp + four softmax warps
        }
        tc::fence_mbar_init();
        tc::tma_prefetch_desc(&tmQ); tc::tma_prefetch_desc(&tmKlin); tc::tma_prefetch_desc(&tmVlin); tc::tma_prefetch_desc(&tmPool);
    }
    if (warp == 1) {
        tc::tmem_alloc(&bars->tmem_slot, kTmemCols);
        tc::tmem_relinquish();
    }
    grid_launch_dependents();
    grid_dependency_wait();                                       // from here on: data of earlier kernels
    if (threadIdx.x == 0) bars->abort_flag = *reinterpret_cast<volatile int *>(err);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const bool live = bars->abort_flag == 0;                      // an earlier kernel gave up: do not pile on

    // Every role walks the same sequence of items: the producer draws an index from the launch's counter and passes it on
    // through a two-slot ring.  `n` counts this CTA's items, `g` its key blocks since the kernel began: the stage of a K / V
    // tile, the S / P buffer of a block and the phase of every barrier follow from g, so the pipelines run on across items.
    // take_item(n): the index of this CTA's n-th item, or -1 when the list is exhausted (consumer side of the ring).
    auto take_item = [&](int n, bool &ok) {
        const int slot = n & 1;
        ok = __all_sync(0xffffffffu, tc::mbar_wait(&bars->item_full[slot], (n >> 1) & 1, err));
        const int idx = ok ? bars->ring[slot] : -1;
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&bars->item_empty[slot]);
        return idx;
    };

    if (!live) {
    } else if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int g = 0;
            for (int n = 0;; ++n) {
                const int slot = n & 1;
                if (!tc::mbar_wait(&bars->item_empty[slot], ((n >> 1) & 1) ^ 1, err)) break;
                int idx = atomicAdd(next_item, 1);
                if (idx >= n_items) idx = -1;
                bars->ring[slot] = idx;
                tc::mbar_arrive(&bars->item_full[slot]);
                if (idx < 0) break;
                const AttnItem it = items[idx];
                const SeqDesc sd = seqs[it.seq];
                const int nb = it.blk1 - it.blk0;
                int d0, n_diag;
                own_key_blocks(it, sd, d0, n_diag);
                const int n_paged_blocks = (sd.n_paged + kKeys - 1) / kKeys;      // = the user's page count
                if (!tc::mbar_wait(&bars->q_empty, (n & 1) ^ 1, err)) break;       // the previous item's last Q K^T has read Q
                tc::mbar_expect_tx(&bars->q_full, kQBytes);
                tc::tma_load_2d(sQ, &tmQ, it.head * kDh, sd.q_row0 + it.q0, &bars->q_full);
                bool ok = true;
                for (int j = 0; j < nb + n_diag; ++j, ++g) {
                    const int b = it.blk0 + j;
                    const int s = g % kStagesKV;
                    const uint32_t par = ((g / kStagesKV) & 1) ^ 1;
                    int ky, vy;
                    const CUtensorMap *mk, *mv;
                    if (j >= nb) {                                       // the candidates' own rows
                        ky = vy = sd.self_row0 + it.q0 + (d0 + j - nb) * kKeys;
                        mk = &tmKlin; mv = &tmVlin;
                    } else if (b < n_paged_blocks) {
                        const int page = pt[sd.pt_base + b];
                        ky = ((page * n_layers + layer) * 2) * 64; vy = ky + 64;
                        mk = &tmPool; mv = &tmPool;
                    } else {
                        ky = vy = sd.lin_row0 + (b - n_paged_blocks) * kKeys;
                        mk = &tmKlin; mv = &tmVlin;
                    }
                    if (!(ok = tc::mbar_wait(&bars->k_empty[s], par, err))) break;
                    tc::mbar_expect_tx(&bars->k_full[s], kKVBytes);
                    tc::tma_load_2d(sK + s * kKVBytes, mk, it.head * kDh, ky, &bars->k_full[s]);
                    if (!(ok = tc::mbar_wait(&bars->v_empty[s], par, err))) break;
                    tc::mbar_expect_tx(&bars->v_full[s], kKVBytes);
                    tc::tma_load_2d(sV + s * kKVBytes, mv, it.head * kDh, vy, &bars->v_full[s]);
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (the whole warp walks the loop so
        // that addresses and descriptors stay warp-uniform; one elected lane issues the tcgen05 instructions)
        constexpr uint32_t idesc_qk = tc::make_idesc(128, kKeys, 0, 0);   // Q, K both K-major
        constexpr uint32_t idesc_pv = tc::make_idesc(128, kDh, 0, 1);     // P from TMEM, V MN-major
        const uint64_t qdesc = tc::smem_desc_sw128(tc::smem_u32(sQ));
        int g = 0;
        bool ok = true;
        for (int n = 0; ok; ++n) {
            const int idx = take_item(n, ok);
            if (idx < 0) break;
            const AttnItem it = items[idx];
            int d0, n_diag;
            own_key_blocks(it, seqs[it.seq], d0, n_diag);
            const int nb = it.blk1 - it.blk0 + n_diag;         // key blocks of the item, the candidates' own included
            ok = tc::mbar_wait(&bars->q_full, n & 1, err);
            if (!ok) break;
            auto issue_qk = [&](int j) {        // S[(g + j) & 1] = Q K(j)^T; the item's last one also hands Q back
                const int gb = g + j, s = gb % kStagesKV, b = gb & 1;
                if (!tc::mbar_wait(&bars->k_full[s], (gb / kStagesKV) & 1, err)) return false;
                tc::tc_fence_after();
                const uint64_t kdesc = tc::smem_desc_sw128(tc::smem_u32(sK + s * kKVBytes));
                if (tc::elect_one()) {
#pragma unroll
                    for (int k = 0; k < kDh / 16; ++k)
                        tc::mma_ss(tmem_base + kColS + b * kKeys, qdesc + 2 * k, kdesc + 2 * k, idesc_qk, k != 0);
                    tc::mma_commit(&bars->s_full[b]);
                    tc::mma_commit(&bars->k_empty[s]);
                    if (j == nb - 1) tc::mma_commit(&bars->q_empty);
                }
                __syncwarp();
                return true;
            };
            // Both S buffers are free here: every P V of the previous item has been issued, each of them after the softmax
            // threads had taken the S of its block into registers.
            if (nb == 0) {
                if (lane == 0) tc::mbar_arrive(&bars->q_empty);
                __syncwarp();
            }
            if (nb > 0) ok = issue_qk(0);
            if (ok && nb > 1) ok = issue_qk(1);
            for (int j = 0; j < nb && ok; ++j) {
                const int gb = g + j, s = gb % kStagesKV, b = gb & 1;
                if (!(ok = tc::mbar_wait(&bars->p_full[b], (gb >> 1) & 1, err))) break;
                if (!(ok = tc::mbar_wait(&bars->v_full[s], (gb / kStagesKV) & 1, err))) break;
                tc::tc_fence_after();
                const uint64_t vdesc = tc::smem_desc_sw128(tc::smem_u32(sV + s * kKVBytes));
                if (tc::elect_one()) {
#pragma unroll
                    for (int k = 0; k < kKeys / 16; ++k)      // 16 keys per instruction: 8 TMEM columns of P, 2048 bytes of V
                        tc::mma_ts(tmem_base + kColO, tmem_base + kColP + b * (kKeys / 2) + 8 * k, vdesc + 128 * k, idesc_pv, (j | k) != 0);
                    tc::mma_commit(&bars->p_free[b]);          // P[b] consumed; also "O holds blocks 0..j of the item"
                    tc::mma_commit(&bars->v_empty[s]);
                }
                __syncwarp();
                // QK(j + 2) follows PV(j) in issue order, and a commit covers everything issued before it: a softmax
                // thread that sees s_full of block j + 2 also knows that P[b] has been consumed.  S[b] is free as well:
                // P(j) was published only after the softmax had taken S(j) into registers.  (The first P V of the next
                // item overwrites O: it waits for that item's first P, which every softmax thread publishes only after
                // its epilogue has read O.)
                if (j + 2 < nb) ok = issue_qk(j + 2);
            }
            g += nb;
        }
    } else {
        // ---------------------------------------------------------------- softmax / correction / epilogue
        const int quad = warp & 3;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const float c = 0.125f * 1.4426950408889634f;        // 1/sqrt(64) * log2(e)
        int g = 0;
        bool ok = true;
        for (int n = 0; ok; ++n) {
        const int idx = take_item(n, ok);
        if (idx < 0) break;
        const AttnItem it = items[idx];
        const SeqDesc sd = seqs[it.seq];
        int d0, n_diag;
        own_key_blocks(it, sd, d0, n_diag);
        const int nb_keys = it.blk1 - it.blk0, nb = nb_keys + n_diag;     // the candidates' own keys come last
        const int n_paged_blocks = (sd.n_paged + kKeys - 1) / kKeys;      // = the user's page count
        const int r = quad * 32 + lane;                      // row of the tile this thread owns
        const int tpos = sd.q_pos0 + it.q0 + r;              // sequence position of the row
        const bool is_cand = tpos >= sd.causal_end;
        const int lim = is_cand ? sd.causal_end - 1 : tpos;  // last visible key position
        const int tile_min_lim = (sd.q_pos0 + it.q0 >= sd.causal_end) ? sd.causal_end - 1 : sd.q_pos0 + it.q0;
        // Blocks [0, n_clean) of the user are complete (64 keys) and visible to every row of the tile: no mask, and none of
        // the per-block position arithmetic, which otherwise sits as a dependent chain between publishing P(j) and polling
        // for S(j + 1).  Pages come first in the block order, then the 64-row groups of linear keys.
        int n_clean = min(sd.n_paged / kKeys, (tile_min_lim + 1) / kKeys);
        if (n_clean == n_paged_blocks && tile_min_lim >= sd.lin_pos0) n_clean += min(sd.n_lin, tile_min_lim + 1 - sd.lin_pos0) / kKeys;
        n_clean -= it.blk0;                                   // relative to the item's first block
        float m = -INFINITY, l = 0.f;
        // a warp whose 32 rows all lie past the tile's last row keeps the hand-shakes going but takes no exponentials:
        // its rows of P (and of O) hold whatever TMEM held, which only ever reaches those same, unused, rows
        const bool warp_live = quad * 32 < it.n_q;

        for (int j = 0; j < nb && ok; ++j) {
            const int gb = g + j, b = gb & 1;
            const bool own_keys = j >= nb_keys;              // a block of the candidates' own keys
            bool need_mask = false;
            int jmax = kKeys;                                // keys jj < jmax of this block are visible to this row
            if (j >= n_clean && !own_keys) {
                const int blk = it.blk0 + j;
                const bool paged = blk < n_paged_blocks;
                const int kidx0 = paged ? blk * kKeys : (blk - n_paged_blocks) * kKeys;    // index of the block's first key in its source
                const int kpos0 = paged ? kidx0 : sd.lin_pos0 + kidx0;                     // its sequence position
                const int n_valid = min(kKeys, (paged ? sd.n_paged : sd.n_lin) - kidx0);
                need_mask = (n_valid < kKeys) || (kpos0 + kKeys - 1 > tile_min_lim);
                jmax = min(n_valid, lim - kpos0 + 1);
            }

            ok = __all_sync(0xffffffffu, tc::mbar_wait(&bars->s_full[b], (gb >> 1) & 1, err));
            if (!ok) break;
            tc::tc_fence_after();
            if (!warp_live) {
                tc::tc_fence_before();
                tc::mbar_arrive(&bars->p_full[b]);
                continue;
            }

            // the S row of this block, in registers
            uint32_t s0[32], s1[32];
            tc::tmem_ld32(lane_addr + kColS + b * kKeys, s0);
            tc::tmem_ld32(lane_addr + kColS + b * kKeys + 32, s1);
            tc::tmem_ld_wait();                              // (S[b] is handed back with P(j): see the MMA issuer)
            if (need_mask) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (i >= jmax) s0[i] = kPointwise ? 0u : 0xff800000u;      // -inf (softmax) or a logit of 0: SiLU(0) = 0
                    if (32 + i >= jmax) s1[i] = kPointwise ? 0u : 0xff800000u;
                }
            }
            if (own_keys) {
                // a candidate row of this 64-row group sees its own key (the diagonal of the block) and nothing else;
                // every other row of the tile sees nothing here
                const int own = is_cand ? r - (d0 + j - nb_keys) * kKeys : -1;
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    s0[i] = select_eq(i, own, s0[i], kPointwise ? 0u : 0xff800000u);
                    s1[i] = select_eq(32 + i, own, s1[i], kPointwise ? 0u : 0xff800000u);
                }
            }
            if constexpr (kPointwise) {
                // p = SiLU(z) = h + h tanh(h), h = z / 2, z = s / sqrt(d_h): one MUFU op per key, bf16 P into TMEM
                const uint64_t hc2 = pack2(0.0625f, 0.0625f), zero2 = pack2(0.f, 0.f);
                uint32_t pk[16];
#pragma unroll
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const uint32_t a0 = half == 0 ? s0[2 * i] : s1[2 * i], a1 = half == 0 ? s0[2 * i + 1] : s1[2 * i + 1];
                        float h0, h1, t0, t1, p0, p1;
                        const uint64_t h2 = fma2(pack2(__uint_as_float(a0), __uint_as_float(a1)), hc2, zero2);
                        unpack2(h2, h0, h1);
                        asm("tanh.approx.f32 %0, %1;" : "=f"(t0) : "f"(h0));
                        asm("tanh.approx.f32 %0, %1;" : "=f"(t1) : "f"(h1));
                        unpack2(fma2(h2, pack2(t0, t1), h2), p0, p1);
                        pk[i] = tc::pack_bf16(p0, p1);
                    }
                    tc::tmem_st16(lane_addr + kColP + b * (kKeys / 2) + 16 * half, pk);
                }
                tc::tmem_st_wait();
                tc::tc_fence_before();
                tc::mbar_arrive(&bars->p_full[b]);
                continue;
            }
            // p = 2^(s c - m c), bf16 P into TMEM (P[b] is free: see the MMA issuer), row sum in fp32.  The exponentials
            // are first taken against the running maximum as it stood before this block; only if the row sum shows that
            // some p may have exceeded 2^8 (or the row has no maximum yet) is the block maximum computed, the running
            // maximum raised, O rescaled and the block redone.  No maximum is on the fast path.
            // Every fourth pair takes its exponentials on the FMA pipe instead (exp2_fma_pipe): the XU pipe is what the two
            // CTAs of an SM compete for (measured: 5-7 % off a rank launch; an eighth or three eighths gain less).  (A compile-time pattern: a run-time switch between the two forms inside
            // the unrolled block cost more than the off-loading gains.)
            auto exp_block = [&](float mc) {
                const uint64_t c2 = pack2(c, c), nmc2 = pack2(-mc, -mc);
                uint64_t ra = pack2(0.f, 0.f), rb = ra;
                uint32_t pk[16];
#pragma unroll
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        const uint32_t a0 = half == 0 ? s0[2 * i] : s1[2 * i], a1 = half == 0 ? s0[2 * i + 1] : s1[2 * i + 1];
                        const uint32_t a2 = half == 0 ? s0[2 * i + 2] : s1[2 * i + 2], a3 = half == 0 ? s0[2 * i + 3] : s1[2 * i + 3];
                        const uint64_t xa = fma2(pack2(__uint_as_float(a0), __uint_as_float(a1)), c2, nmc2);
                        const uint64_t xb = fma2(pack2(__uint_as_float(a2), __uint_as_float(a3)), c2, nmc2);
                        float p0, p1, p2, p3, x0, x1, x2, x3;
                        unpack2(xb, x2, x3);
                        p2 = ex2(x2); p3 = ex2(x3);
                        if (kOffload && (i & 2) != 0) {
                            exp2_fma_pipe(xa, p0, p1);
                        } else {
                            unpack2(xa, x0, x1);
                            p0 = ex2(x0); p1 = ex2(x1);
                        }
                        ra = add2(ra, pack2(p0, p1)); rb = add2(rb, pack2(p2, p3));
                        pk[i] = tc::pack_bf16(p0, p1); pk[i + 1] = tc::pack_bf16(p2, p3);
                    }
                    tc::tmem_st16(lane_addr + kColP + b * (kKeys / 2) + 16 * half, pk);
                }
                float r0, r1;
                unpack2(add2(ra, rb), r0, r1);
                return r0 + r1;
            };
            float rs = 0.f, alpha = 1.f;
            bool redo = true;
            if (j > 0) {
                rs = exp_block((m == -INFINITY) ? 0.f : m * c);
                redo = __any_sync(0xffffffffu, !(rs <= kRowSumLimit) || m == -INFINITY);
            }
            if (redo) {
                float mx = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    mx = max3(mx, __uint_as_float(s0[i]), __uint_as_float(s0[i + 1]));
                    mx1 = max3(mx1, __uint_as_float(s0[i + 2]), __uint_as_float(s0[i + 3]));
                    mx2 = max3(mx2, __uint_as_float(s1[i]), __uint_as_float(s1[i + 1]));
                    mx3 = max3(mx3, __uint_as_float(s1[i + 2]), __uint_as_float(s1[i + 3]));
                }
                mx = fmaxf(fmaxf(mx, mx1), fmaxf(mx2, mx3));
                const bool raise = mx > m;                    // false when mx == -inf
                if (raise) {
                    alpha = (m == -INFINITY) ? 0.f : ex2((m - mx) * c);
                    m = mx;
                }
                if (j > 0 && __any_sync(0xffffffffu, raise)) {
                    // correction: O must hold blocks 0..j-1 completely before it is rescaled
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&bars->p_free[(gb - 1) & 1], ((gb - 1) >> 1) & 1, err));
                    if (!ok) break;
                    tc::tc_fence_after();
#pragma unroll 1
                    for (int cc = 0; cc < kDh; cc += 16) {
                        uint32_t ov[16];
                        tc::tmem_ld16(lane_addr + kColO + cc, ov);
                        tc::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 16; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                        tc::tmem_st16(lane_addr + kColO + cc, ov);
                    }
                }
                rs = exp_block((m == -INFINITY) ? 0.f : m * c);
            }
            l = fmaf(l, alpha, rs);
            tc::tmem_st_wait();
            tc::tc_fence_before();
            tc::mbar_arrive(&bars->p_full[b]);     // P(j) (and any correction of O) is in TMEM
        }

        if (!ok) break;
        // ---- epilogue: O / l, or the split partial
        if (nb > 0) ok = __all_sync(0xffffffffu, tc::mbar_wait(&bars->p_free[(g + nb - 1) & 1], ((g + nb - 1) >> 1) & 1, err));
        if (!ok) break;
        tc::tc_fence_after();
        if (ok && warp_live) {
            float o[kDh];
            if (nb > 0) {
#pragma unroll
                for (int cc = 0; cc < kDh; cc += 16) {
                    uint32_t ov[16];
                    tc::tmem_ld16(lane_addr + kColO + cc, ov);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[cc + i] = __uint_as_float(ov[i]);
                }
            } else {
#pragma unroll
                for (int i = 0; i < kDh; ++i) o[i] = 0.f;
            }
            const bool row_ok = r < it.n_q;
            const int64_t row = (int64_t)sd.q_row0 + it.q0 + r;
            if constexpr (kPointwise) {
                // the normaliser is the number of keys the row may see (every key position below its limit, plus itself for
                // a candidate); a split item hands it over as l with m = 0, so that the merge of partials needs no change
                const float n_seen = (float)(is_cand ? sd.causal_end + 1 : tpos + 1);
                m = 0.f;
                l = (it.partial_slot < 0 || it.blk0 == 0) ? n_seen : 0.f;
            }
            if (row_ok) {
                if (it.partial_slot < 0) {
                    const float inv = 1.f / l;
                    uint4 *dst = reinterpret_cast<uint4 *>(out + row * d_model + it.head * kDh);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        uint4 w4;
                        w4.x = tc::pack_bf16(o[8 * i] * inv, o[8 * i + 1] * inv);
                        w4.y = tc::pack_bf16(o[8 * i + 2] * inv, o[8 * i + 3] * inv);
                        w4.z = tc::pack_bf16(o[8 * i + 4] * inv, o[8 * i + 5] * inv);
                        w4.w = tc::pack_bf16(o[8 * i + 6] * inv, o[8 * i + 7] * inv);
                        dst[i] = w4;
                    }
                } else {
                    float4 *dst = reinterpret_cast<float4 *>(partial + ((size_t)it.partial_slot * kQTile + r) * kPartStride);
                    dst[0] = make_float4(m, l, 0.f, 0.f);
#pragma unroll
                    for (int i = 0; i < kDh / 4; ++i) dst[1 + i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                }
            }
        }
        g += nb;
        }   // items
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem_base, kTmemCols);
}

// Combine the (m, l, O) partials of a split work item:  O = sum_i 2^((m_i - M) c) O_i / sum_i 2^((m_i - M) c) l_i.
// blockIdx.x = item, blockIdx.y = group of 8 rows; one warp per row, a lane per pair of output columns: every load is a
// coalesced row segment and all rows are in flight at once (the kernel is a chain of two memory round trips).
__global__ void __launch_bounds__(256)
attention_merge_kernel(const AttnMerge *__restrict__ merges, const SeqDesc *__restrict__ seqs, const float *__restrict__ partial,
                       int d_model, __nv_bfloat16 *__restrict__ out)
{
    grid_launch_dependents();
    grid_dependency_wait();
    const AttnMerge mg = merges[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float c = 0.125f * 1.4426950408889634f;
    const int64_t row0 = (int64_t)seqs[mg.seq].q_row0 + mg.q0;
    const int r = blockIdx.y * 8 + warp;
    if (r < mg.n_q) {
        float M = -INFINITY;
        for (int i = 0; i < mg.n_splits; ++i) M = fmaxf(M, partial[((size_t)(mg.slot0 + i) * kQTile + r) * kPartStride]);
        float o0 = 0.f, o1 = 0.f, l = 0.f;
        for (int i = 0; i < mg.n_splits; ++i) {
            const float *p = partial + ((size_t)(mg.slot0 + i) * kQTile + r) * kPartStride;
            const float mi = p[0];
            const float wgt = (mi == -INFINITY) ? 0.f : ex2((mi - M) * c);
            const float2 v = *reinterpret_cast<const float2 *>(p + 4 + 2 * lane);
            l = fmaf(p[1], wgt, l);
            o0 = fmaf(v.x, wgt, o0);
            o1 = fmaf(v.y, wgt, o1);
        }
        const float inv = 1.f / l;
        *reinterpret_cast<uint32_t *>(out + (row0 + r) * d_model + mg.head * kDh + 2 * lane) = tc::pack_bf16(o0 * inv, o1 * inv);
    }
}

}  // namespace

cudaError_t launch_attention_tc(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV, const CUtensorMap &tmPool,
                                const AttnItem *items, int n_items, const AttnMerge *merges, int n_merges, const SeqDesc *seqs,
                                const int32_t *pt, int n_layers, int layer, int d_model, int attn_kind, __nv_bfloat16 *out,
                                float *partial, int *next_item, int n_sms, int *err, cudaStream_t stream, int64_t *launches)
{
    if (n_items == 0) return cudaSuccess;
    static PerDeviceValue attr_set;
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (!attr_set.get(dev)) {
        cudaError_t e = cudaFuncSetAttribute(attention_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attention_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set.set(dev, 1);
    }
    *launches += 1;
    auto kernel = attn_kind == ATTN_POINTWISE ? attention_tc_kernel<true> : attention_tc_kernel<false>;
    const int grid = std::min(n_items, 2 * std::max(1, n_sms));       // two CTAs per SM, each drawing items until none is left
    cudaError_t e = launch_dependent(kernel, dim3(grid), dim3(192), (size_t)kSmemBytes, stream, 1, tmQ, tmK, tmV, tmPool, items,
                                     n_items, next_item, seqs, pt, n_layers, layer, d_model, out, partial, err);
    if (e != cudaSuccess || n_merges == 0) return e;
    *launches += 1;
    return launch_dependent(attention_merge_kernel, dim3(n_merges, kQTile / 8), dim3(256), 0, stream, 1, merges, seqs, partial, d_model, out);
}

}  // namespace relaygr

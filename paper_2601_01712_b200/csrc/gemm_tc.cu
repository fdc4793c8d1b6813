// bf16 GEMM on the 5th-generation tensor cores: C[m, n] = sum_k A[m, k] W[n, k] with fp32
// accumulators in TMEM.  The K extents of this model are short (d_model or d_ff), so a tile's
// mainloop is a handful of MMAs and the epilogue - reading the accumulators back and moving
// them to global memory - weighs as much.  The kernel is therefore persistent (one CTA, or one
// CTA pair, per SM or SM pair walks a list of output tiles) with two accumulators in TMEM, so
// that the epilogue of one tile runs under the TMA loads and MMAs of the next, and the
// epilogue hands its output to the TMA unit: a warp stages 32 rows x 128 bytes in shared
// memory (128-byte swizzle, conflict-free) and one lane issues a bulk tensor store - or, for
// the residual stream, a bulk fp32 add-reduction (x += tile, performed in L2: the residual
// never travels to the SM).  K/V rows of a pre-infer call go straight into the users' pages:
// with one bulk tensor store where a warp's 32 rows are 32 consecutive slots of one page,
// with plain stores after a page-table walk per row otherwise.
//
// Two shapes (Cfg below): single CTAs with 128 x 128 tiles, and CTA pairs (a cluster of two,
// tcgen05 cta_group::2) with 256 x 256 tiles, where each CTA loads its 128 rows of A and half
// of W and the even CTA issues the MMAs for both.
//
// Warp roles (320 threads per CTA): warp 0 = TMA producer (128 x 64 tiles of A and W, 128-byte
// swizzle, five-stage ring), warp 1 = TMEM owner + MMA issuer (tcgen05.mma K16), warps 2-9 =
// epilogue: warp w reads TMEM lanes 32 (w % 4) .. +31 (its hardware quadrant), columns
// (BN / 2) ((w - 2) / 4) .. + BN / 2 - 1, 64 at a time, applies bias / SiLU in the
// row-per-thread layout tcgen05.ld delivers and stages the result for the store.
#include "kernels.cuh"
#include "tc_common.cuh"

namespace relaygr {

namespace {

constexpr int BM = 128, BK = 64, kMaxStages = 5;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kABytes = BM * BK * 2;
constexpr int kPatchBytes = 32 * 128;                                // one staged store: 32 rows x 128 bytes
constexpr int kPatches = 1;                                          // per warp (a store has read its patch long before the next is packed)

// A tile is 128 x BN per CTA.  CTAS = 1: BN = 128 (or 256), the CTA loads all of A and B.  CTAS = 2: a pair of CTAs works on
// 256 x 256 with one tcgen05 cta_group::2 MMA stream issued by the even CTA; each CTA loads its 128 rows of A and half
// (128 rows) of B, so a K block costs each CTA 32 KB of shared-memory writes and 32 KB of operand reads per 512 tensor
// clocks - the shared-memory bandwidth that a single CTA spends on 128 x 128.  The stage ring is as deep as shared
// memory allows.
template <int BN, int CTAS> struct Cfg {
    static constexpr int kBBytes = (BN / CTAS) * BK * 2;
    static constexpr int kStage = kABytes + kBBytes;
    static constexpr int kStages = (CTAS == 1 && BN == 256) ? 3 : 5;
    static constexpr int kOffPatch = kStages * kStage;                                    // 1024-byte aligned: stages are
    static constexpr int kOffBias = kOffPatch + kEpiWarps * kPatches * kPatchBytes;       // per warp BN / 2 floats
    static constexpr int kOffRowOff = kOffBias + kEpiWarps * (BN / 2) * 4;                // per warp 32 x int64
    static constexpr int kOffBars = kOffRowOff + kEpiWarps * 32 * 8;
    static constexpr int kSmemBytes = kOffBars + 256 /*barriers*/ + 1024 /*alignment slack*/;
    static constexpr uint32_t kTmemCols = 2 * BN;
    static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
    static_assert(CTAS == 1 || BN == 256, "a CTA pair works on 256 x 256");
};

struct GemmBars {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[2], acc_empty[2];
    uint32_t tmem_slot;
    int abort_flag;
};
static_assert(sizeof(GemmBars) <= 256, "barrier block");

// 16-byte chunk j of row r of a staged patch (rows of 128 bytes, chunk index XORed with r % 8: the 128-byte swizzle of
// the output tensor maps, and conflict-free for a warp that writes one row per lane)
__device__ __forceinline__ uint4 *patch_chunk(uint8_t *patch, int r, int j)
{
    return reinterpret_cast<uint4 *>(patch + r * 128 + ((j ^ (r & 7)) << 4));
}

// SiLU(z) = z sigmoid(z) = h + h tanh(h), h = z / 2: one MUFU op per element (tanh.approx, relative error 2^-11, below
// the bf16 rounding of the result that follows)
__device__ __forceinline__ float silu(float z)
{
    const float h = 0.5f * z;
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(h));
    return fmaf(h, t, h);
}

template <int BN, int CTAS>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ GemmOutMaps om,
               int64_t M, int N, int K, Epilogue epi, int *err)
{
    using C = Cfg<BN, CTAS>;
    constexpr int STAGES = C::kStages, kStage = C::kStage;
    constexpr uint32_t kTmemCols = C::kTmemCols;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    GemmBars *bars = reinterpret_cast<GemmBars *>(smem + C::kOffBars);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kblocks = K / BK;
    const int n_tiles_n = N / BN;
    const int64_t n_tiles = ((M + BM * CTAS - 1) / (BM * CTAS)) * n_tiles_n;       // tiles of the CTA (or the pair)
    const uint32_t rank = CTAS == 2 ? tc::cluster_ctarank() : 0;                     // this CTA's half of a pair tile
    const int64_t worker = blockIdx.x / CTAS, n_workers = gridDim.x / CTAS;
    const bool leader = rank == 0;                                                   // issues the MMAs, owns full / acc_empty

    // set-up that touches nothing earlier kernels wrote; it may run while the previous kernel is still finishing
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&bars->full[s], 1); tc::mbar_init(&bars->empty[s], 1); }
        for (int s = 0; s < 2; ++s) { tc::mbar_init(&bars->acc_full[s], 1); tc::mbar_init(&bars->acc_empty[s], kEpiWarps * CTAS); }
        tc::fence_mbar_init();
        tc::tma_prefetch_desc(&tmA);
        tc::tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        if constexpr (CTAS == 2) { tc::tmem_alloc_pair(&bars->tmem_slot, kTmemCols); tc::tmem_relinquish_pair(); }
        else { tc::tmem_alloc(&bars->tmem_slot, kTmemCols); tc::tmem_relinquish(); }
    }
    if constexpr (CTAS == 2) tc::cluster_sync();                  // the peer's barriers exist before anything signals them
    grid_launch_dependents();
    grid_dependency_wait();                                       // from here on: data of earlier kernels
    if (threadIdx.x == 0) bars->abort_flag = *reinterpret_cast<volatile int *>(err);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const bool live = bars->abort_flag == 0;                      // an earlier kernel gave up: do not pile on

    if (!live) {
    } else if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer: this CTA's rows of A and of B
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int64_t t = worker; t < n_tiles && ok; t += n_workers) {
                const int m0 = (int)(t / n_tiles_n) * (BM * CTAS) + (int)rank * BM;
                const int n0 = (int)(t % n_tiles_n) * BN + (int)rank * (BN / CTAS);
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    ok = tc::mbar_wait(&bars->empty[s], ((it / STAGES) & 1) ^ 1, err);
                    if (!ok) break;
                    uint8_t *a = smem + s * kStage;
                    if constexpr (CTAS == 2) {
                        // both CTAs' bytes are counted on the even CTA's barrier, which expects the sum
                        if (leader) tc::mbar_expect_tx(&bars->full[s], 2 * kStage);
                        const uint32_t bar = tc::cluster_addr(&bars->full[s], 0);
                        tc::tma_load_2d_pair(a, &tmA, kb * BK, m0, bar);
                        tc::tma_load_2d_pair(a + kABytes, &tmB, kb * BK, n0, bar);
                    } else {
                        tc::mbar_expect_tx(&bars->full[s], kStage);
                        tc::tma_load_2d(a, &tmA, kb * BK, m0, &bars->full[s]);
                        tc::tma_load_2d(a + kABytes, &tmB, kb * BK, n0, &bars->full[s]);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (the whole warp walks the loop so that
        // addresses stay warp-uniform; one elected lane issues the tcgen05 instructions).  In a pair only the even CTA issues.
        if (leader) {
            constexpr uint32_t idesc = tc::make_idesc(BM * CTAS, BN, 0, 0);
            uint32_t it = 0, ti = 0;
            bool ok = true;
            for (int64_t t = worker; t < n_tiles && ok; t += n_workers, ++ti) {
                const uint32_t as = ti & 1;
                ok = tc::mbar_wait(&bars->acc_empty[as], ((ti >> 1) & 1) ^ 1, err);     // the epilogue has drained this accumulator
                if (!ok) break;
                tc::tc_fence_after();
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    ok = tc::mbar_wait(&bars->full[s], (it / STAGES) & 1, err);
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t a = tc::smem_u32(smem + s * kStage);
                    const uint64_t adesc = tc::smem_desc_sw128(a), bdesc = tc::smem_desc_sw128(a + kABytes);
                    if (tc::elect_one()) {
                        // 32 bytes of K per instruction: descriptor start address + 2.  A commit frees the stage (in both
                        // CTAs of a pair) when these MMAs have read it; the last one also hands the accumulator over.
                        if constexpr (CTAS == 2) {
#pragma unroll
                            for (int k = 0; k < BK / 16; ++k)
                                tc::mma_ss_pair(tmem_base + as * BN, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
                            tc::mma_commit_pair(&bars->empty[s], 3);
                            if (kb == kblocks - 1) tc::mma_commit_pair(&bars->acc_full[as], 3);
                        } else {
#pragma unroll
                            for (int k = 0; k < BK / 16; ++k)
                                tc::mma_ss(tmem_base + as * BN, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
                            tc::mma_commit(&bars->empty[s]);
                            if (kb == kblocks - 1) tc::mma_commit(&bars->acc_full[as]);
                        }
                    }
                    __syncwarp();
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue
        const int ew = warp - 2;
        const int quad = warp & 3;                          // TMEM lanes this warp may touch: 32*quad .. 32*quad+31
        const int half = ew >> 2;                           // columns (BN/2)*half .. +BN/2-1 of the tile, 64 at a time
        constexpr int kColsPerWarp = BN / 2;
        uint8_t *patches = smem + C::kOffPatch + ew * (kPatches * kPatchBytes);
        float *bias_s = reinterpret_cast<float *>(smem + C::kOffBias) + ew * kColsPerWarp;
        int64_t *rowoff = reinterpret_cast<int64_t *>(smem + C::kOffRowOff) + ew * 32;
        const bool scatter = epi.mode == EPI_QKV && epi.paged.slab != nullptr;
        uint32_t pp = 0;                                    // the patch the next staged store fills
        // the store that filled this patch last has read it (the one in flight may still read the other patch)
        auto patch_acquire = [&]() -> uint8_t * {
            if (lane == 0) tc::bulk_wait_read<kPatches - 1>();
            __syncwarp();
            return patches + pp * kPatchBytes;
        };
        // every lane has written its row: hand the patch to the TMA unit
        auto patch_submit = [&](const CUtensorMap *map, const uint8_t *patch, int x, int y, bool add) {
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                if (add) tc::tma_reduce_add_2d(map, patch, x, y);
                else tc::tma_store_2d(map, patch, x, y);
                tc::bulk_commit();
            }
            pp ^= (uint32_t)(kPatches - 1);
        };
        uint32_t ti = 0;
        bool ok = true;
        const uint32_t acc_empty_bar = CTAS == 2 ? tc::cluster_addr(&bars->acc_empty[0], 0) : tc::smem_u32(&bars->acc_empty[0]);
        for (int64_t t = worker; t < n_tiles && ok; t += n_workers, ++ti) {
            const int64_t m0 = (t / n_tiles_n) * (BM * CTAS) + rank * BM;
            const int n_w = (int)(t % n_tiles_n) * BN + half * kColsPerWarp;      // first column of this warp's part
            const uint32_t as = ti & 1;
            const int64_t m_base = m0 + quad * 32;
            const int64_t m = m_base + lane;
            // before the accumulator is ready: this warp's slice of the bias, and for K / V rows of a pre-infer call
            // (they go straight into the user's pages) the offset of (page, K, slot) per row
            if (epi.bias) {
#pragma unroll
                for (int c = 0; c < kColsPerWarp; c += 32) bias_s[c + lane] = epi.bias[n_w + c + lane];
            }
            int last_slot = -1, page = 0;
            const bool paged_tile = scatter && epi.col0 + n_w + kColsPerWarp - 1 >= epi.d_model;
            bool run = false;                               // the warp's 32 rows are 32 consecutive slots of one page
            int pool_row0 = 0;                              // row of (page, K, first slot) in the pool map; V is 64 rows on
            if (paged_tile) {
                int64_t off = 0;
                int u = -1, tt = 0;
                if (m < M) {
                    u = find_user(epi.row_off, epi.n_users, (int)m);
                    tt = (int)m - epi.row_off[u];
                    page = epi.paged.pt[epi.seqs[u].pt_base + (tt >> 6)];
                    off = (int64_t)page_elem_offset(epi.paged, page, 0, tt & 63);
                    if (tt == epi.seqs[u].n_q - 1) last_slot = tt & 63;
                }
                rowoff[lane] = off;
                const int u0 = __shfl_sync(0xffffffffu, u, 0), tt0 = __shfl_sync(0xffffffffu, tt, 0), page0 = __shfl_sync(0xffffffffu, page, 0);
                run = __all_sync(0xffffffffu, u >= 0 && u == u0 && tt == tt0 + lane && (tt0 & 63) <= 32);
                pool_row0 = ((page0 * epi.paged.n_layers + epi.paged.layer) * 2) * 64 + (tt0 & 63);
            }
            __syncwarp();
            ok = __all_sync(0xffffffffu, tc::mbar_wait(&bars->acc_full[as], (ti >> 1) & 1, err));
            if (!ok) break;
            tc::tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + as * BN + half * kColsPerWarp;
#pragma unroll 1
            for (int pass = 0; pass < kColsPerWarp / 64; ++pass) {
                uint32_t r0[32], r1[32];
                tc::tmem_ld32(taddr + pass * 64, r0);
                tc::tmem_ld32(taddr + pass * 64 + 32, r1);
                tc::tmem_ld_wait();
                if (pass == kColsPerWarp / 64 - 1) {
                    tc::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {                                          // this warp's part of the accumulator is in registers
                        if constexpr (CTAS == 2) tc::mbar_arrive_cluster(acc_empty_bar + as * 8);
                        else tc::mbar_arrive(&bars->acc_empty[as]);
                    }
                }
                if (m_base >= M) continue;                                       // the whole row group lies past the last row
                const int n = n_w + pass * 64;                                   // first output column of these 64
                if (epi.bias) {
                    const float4 *b4 = reinterpret_cast<const float4 *>(bias_s + pass * 64);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 b = b4[i], c = b4[8 + i];
                        r0[4 * i] = __float_as_uint(__uint_as_float(r0[4 * i]) + b.x);
                        r0[4 * i + 1] = __float_as_uint(__uint_as_float(r0[4 * i + 1]) + b.y);
                        r0[4 * i + 2] = __float_as_uint(__uint_as_float(r0[4 * i + 2]) + b.z);
                        r0[4 * i + 3] = __float_as_uint(__uint_as_float(r0[4 * i + 3]) + b.w);
                        r1[4 * i] = __float_as_uint(__uint_as_float(r1[4 * i]) + c.x);
                        r1[4 * i + 1] = __float_as_uint(__uint_as_float(r1[4 * i + 1]) + c.y);
                        r1[4 * i + 2] = __float_as_uint(__uint_as_float(r1[4 * i + 2]) + c.z);
                        r1[4 * i + 3] = __float_as_uint(__uint_as_float(r1[4 * i + 3]) + c.w);
                    }
                }
                if (epi.mode == EPI_RESID) {
                    // x[m, n .. n+63] += tile, as two fp32 patches of 32 columns
#pragma unroll
                    for (int cc = 0; cc < 2; ++cc) {
                        uint8_t *patch = patch_acquire();
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *patch_chunk(patch, lane, j) = cc == 0 ? make_uint4(r0[4 * j], r0[4 * j + 1], r0[4 * j + 2], r0[4 * j + 3])
                                                                   : make_uint4(r1[4 * j], r1[4 * j + 1], r1[4 * j + 2], r1[4 * j + 3]);
                        patch_submit(&om.o[0], patch, n + cc * 32, (int)m_base, true);
                    }
                    continue;
                }
                if (epi.mode == EPI_STORE && epi.silu) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        r0[i] = __float_as_uint(silu(__uint_as_float(r0[i])));
                        r1[i] = __float_as_uint(silu(__uint_as_float(r1[i])));
                    }
                }
                // bf16 outputs: 64 columns = one 128-byte row per lane
                int which = 0, c = n;                                            // destination tensor and its column
                if (epi.mode == EPI_QKV) {
                    const int col = epi.col0 + n;
                    which = (col >= epi.d_model) + (col >= 2 * epi.d_model); c = col - which * epi.d_model;
                }
                const bool paged = paged_tile && which > 0;
                uint8_t *patch;
                if (paged && !run) {
                    if (lane == 0) tc::bulk_wait_read<0>();                      // the patches are idle: this path reads its own staging
                    __syncwarp();
                    patch = patches;
                } else {
                    patch = patch_acquire();
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    *patch_chunk(patch, lane, j) =
                        make_uint4(tc::pack_bf16(__uint_as_float(r0[8 * j]), __uint_as_float(r0[8 * j + 1])),
                                   tc::pack_bf16(__uint_as_float(r0[8 * j + 2]), __uint_as_float(r0[8 * j + 3])),
                                   tc::pack_bf16(__uint_as_float(r0[8 * j + 4]), __uint_as_float(r0[8 * j + 5])),
                                   tc::pack_bf16(__uint_as_float(r0[8 * j + 6]), __uint_as_float(r0[8 * j + 7])));
                    *patch_chunk(patch, lane, 4 + j) =
                        make_uint4(tc::pack_bf16(__uint_as_float(r1[8 * j]), __uint_as_float(r1[8 * j + 1])),
                                   tc::pack_bf16(__uint_as_float(r1[8 * j + 2]), __uint_as_float(r1[8 * j + 3])),
                                   tc::pack_bf16(__uint_as_float(r1[8 * j + 4]), __uint_as_float(r1[8 * j + 5])),
                                   tc::pack_bf16(__uint_as_float(r1[8 * j + 6]), __uint_as_float(r1[8 * j + 7])));
                }
                if (!paged) {
                    patch_submit(&om.o[which], patch, c, (int)m_base, false);
                    continue;
                }
                if (run) {
                    // the 32 rows are consecutive slots of one page: one bulk tensor store into the pool
                    patch_submit(&om.pool, patch, c, pool_row0 + (which - 1) * 64, false);
                } else {
                // K / V rows into pages: 8 lanes per row copy its 128 bytes to (page, K | V, slot)
                __syncwarp();
                __nv_bfloat16 *kv = reinterpret_cast<__nv_bfloat16 *>(epi.paged.slab) + (size_t)(which - 1) * 64 * epi.d_model + c;
                const int rr = lane >> 3, cj = lane & 7;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const int r = it * 4 + rr;
                    if (m_base + r < M) *reinterpret_cast<uint4 *>(kv + rowoff[r] + cj * 8) = *patch_chunk(patch, r, cj);
                }
                __syncwarp();
                }
                if (last_slot >= 0 && last_slot < 63) {
                    // last prefix row of a user: clear the unused slots of its last page (they are masked, but must hold finite values)
                    __nv_bfloat16 *slab = reinterpret_cast<__nv_bfloat16 *>(epi.paged.slab);
                    const uint4 z = make_uint4(0, 0, 0, 0);
                    for (int s = last_slot + 1; s < 64; ++s) {
                        uint4 *zp = reinterpret_cast<uint4 *>(slab + page_elem_offset(epi.paged, page, which - 1, s) + c);
#pragma unroll
                        for (int j = 0; j < 8; ++j) zp[j] = z;
                    }
                }
            }
        }
        if (lane == 0) tc::bulk_wait_read<0>();             // the patch has been read; the grid's completion covers the global writes
    }
    tc::tc_fence_before();
    __syncthreads();
    if constexpr (CTAS == 2) {
        tc::cluster_sync();                                       // the peer no longer signals this CTA's barriers or uses its operands
        if (warp == 1) tc::tmem_dealloc_pair(tmem_base, kTmemCols);
    } else {
        if (warp == 1) tc::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

template <int BN, int CTAS>
static cudaError_t launch_cfg(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmOutMaps &om, int64_t M, int N, int K,
                              const Epilogue &epi, int *err, cudaStream_t stream)
{
    using C = Cfg<BN, CTAS>;
    static PerDeviceValue workers_of;               // CTAs (or CTA pairs) that can be resident at once: one per SM (or SM pair)
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    int n_workers_max = workers_of.get(dev);
    if (n_workers_max == 0) {
        int n_sms = 0;
        e = cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<BN, CTAS>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
        int n = n_sms / CTAS;
        if (e == cudaSuccess && CTAS == 2) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)(2 * n)); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = C::kSmemBytes;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int max_clusters = 0;
            e = cudaOccupancyMaxActiveClusters(&max_clusters, gemm_tc_kernel<BN, CTAS>, &cfg);
            if (e == cudaSuccess && max_clusters < n) n = max_clusters;
        }
        if (e != cudaSuccess) return e;
        if (n < 1) return cudaErrorLaunchOutOfResources;
        n_workers_max = n;
        workers_of.set(dev, n);
    }
    const int64_t tiles = ((M + BM * CTAS - 1) / (BM * CTAS)) * (N / BN);
    const unsigned workers = (unsigned)(tiles < n_workers_max ? tiles : n_workers_max);
    return launch_dependent(gemm_tc_kernel<BN, CTAS>, dim3(workers * CTAS), dim3(kThreads), (size_t)C::kSmemBytes, stream, CTAS, tmA, tmB, om,
                            M, N, K, epi, err);
}

cudaError_t launch_gemm_tc(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmOutMaps &om, int64_t M, int N, int K,
                           const Epilogue &epi, int *err, cudaStream_t stream, int64_t *launches)
{
    if (M == 0 || N == 0) return cudaSuccess;
    *launches += 1;
    return gemm_pair(M, N, K) ? launch_cfg<256, 2>(tmA, tmB, om, M, N, K, epi, err, stream)
                        : launch_cfg<128, 1>(tmA, tmB, om, M, N, K, epi, err, stream);
}

}  // namespace relaygr

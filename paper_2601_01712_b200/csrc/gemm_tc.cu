// bf16 GEMM on the 5th-generation tensor cores: C[m, n] = sum_k A[m, k] W[n, k] with fp32
// accumulators in TMEM.  The K extents of this model are short (d_model or d_ff), so a tile's
// mainloop is a handful of MMAs and the epilogue - reading 128 x 128 accumulators back and
// moving them to global memory - is the longer half.  The kernel is therefore persistent
// (one CTA per SM walks a list of 128 x 128 output tiles) with two accumulators in TMEM, so
// that the epilogue of one tile runs under the TMA loads and MMAs of the next, and the
// epilogue goes through shared memory so that every global access is a full row segment.
//
// Warp roles (320 threads): warp 0 = TMA producer (128 x 64 tiles of A and W, 128-byte
// swizzle, 4-stage ring), warp 1 = TMEM owner + MMA issuer (tcgen05.mma M128 N128 K16),
// warps 2-9 = epilogue: warp w reads TMEM lanes 32 (w % 4) .. +31 (its hardware quadrant),
// columns 64 ((w - 2) / 4) .. +63 in two chunks of 32, applies bias / SiLU in the
// row-per-thread layout tcgen05.ld delivers, transposes the chunk through a private
// shared-memory patch and then reads / writes global memory with 8 (fp32) or 4 (bf16)
// lanes per row.
#include "kernels.cuh"
#include "tc_common.cuh"

namespace relaygr {

namespace {

constexpr int BM = 128, BK = 64, kMaxStages = 4;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kABytes = BM * BK * 2;
constexpr int kPatchPitchF32 = 36;                                  // floats per staged row (32 + 4 pad): conflict-free float4 access
constexpr int kPatchBytes = 32 * kPatchPitchF32 * 4;                // 4608 B per warp

// Tile width BN: 128, or 256 for long mainloops (gemm_tile_n).  The stage ring is as deep as shared memory allows.
template <int BN> struct Cfg {
    static constexpr int kBBytes = BN * BK * 2;
    static constexpr int kStage = kABytes + kBBytes;
    static constexpr int kStages = BN == 256 ? 3 : 4;
    static constexpr int kSmemBytes = kStages * kStage + kEpiWarps * kPatchBytes + kEpiWarps * 32 * 8 /*row offsets*/ + 256 /*barriers*/ +
                                      1024 /*alignment slack*/;
    static constexpr uint32_t kTmemCols = 2 * BN;
};

struct GemmBars {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[2], acc_empty[2];
    uint32_t tmem_slot;
    int abort_flag;
};

// One 32-row x 32-column chunk of the accumulator tile, held one row per lane in v[32].
// m_base = first row of the warp's quadrant, n = first global output column of the chunk.
__device__ __forceinline__ void epilogue_chunk(const Epilogue &e, int64_t m_base, int64_t M, int n, int N, float (&v)[32], int lane,
                                               float *patch, const int64_t *rowoff)
{
    if (e.bias) {
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
            const float4 b = *reinterpret_cast<const float4 *>(e.bias + n + i);
            v[i] += b.x; v[i + 1] += b.y; v[i + 2] += b.z; v[i + 3] += b.w;
        }
    }
    if (e.mode == EPI_RESID) {
        // stage fp32, then 8 lanes per row: x[m, n .. n+31] += chunk
        float4 *prow = reinterpret_cast<float4 *>(patch + lane * kPatchPitchF32);
#pragma unroll
        for (int i = 0; i < 8; ++i) prow[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        __syncwarp();
        const int rr = lane >> 3, c4 = (lane & 7) * 4;
        float4 x[8];
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int64_t m = m_base + it * 4 + rr;
            x[it] = m < M ? *reinterpret_cast<const float4 *>(e.resid + m * N + n + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int r = it * 4 + rr;
            const int64_t m = m_base + r;
            const float4 t = *reinterpret_cast<const float4 *>(patch + r * kPatchPitchF32 + c4);
            if (m < M) *reinterpret_cast<float4 *>(e.out_f32 + m * N + n + c4) = make_float4(x[it].x + t.x, x[it].y + t.y, x[it].z + t.z, x[it].w + t.w);
        }
        __syncwarp();
        return;
    }
    if (e.mode == EPI_STORE && e.silu) {
        // SiLU(z) = z sigmoid(z) = h + h tanh(h), h = z / 2: one MUFU op per element (tanh.approx, relative error 2^-11,
        // below the bf16 rounding of the result that follows)
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float h = 0.5f * v[i];
            float t;
            asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(h));
            v[i] = fmaf(h, t, h);
        }
    }
    // bf16 outputs: stage 64-byte rows (pitch 80 bytes), then 4 lanes per row write 16 bytes each
    constexpr int kPitchB = 80;
    uint8_t *pb = reinterpret_cast<uint8_t *>(patch);
    uint4 *prow = reinterpret_cast<uint4 *>(pb + lane * kPitchB);
#pragma unroll
    for (int i = 0; i < 4; ++i)
        prow[i] = make_uint4(tc::pack_bf16(v[8 * i], v[8 * i + 1]), tc::pack_bf16(v[8 * i + 2], v[8 * i + 3]),
                             tc::pack_bf16(v[8 * i + 4], v[8 * i + 5]), tc::pack_bf16(v[8 * i + 6], v[8 * i + 7]));
    __syncwarp();
    // where the chunk's rows go
    __nv_bfloat16 *base;          // element (row 0 of the call, column c of this chunk)
    int64_t pitch;                // elements between rows of the call (unused for the paged scatter)
    bool paged = false;
    int which = 0, c = n;
    if (e.mode == EPI_STORE) {
        base = reinterpret_cast<__nv_bfloat16 *>(e.out) + n; pitch = N;
    } else {
        const int col = e.col0 + n, d = e.d_model;
        which = col / d; c = col - which * d;
        pitch = d;
        if (which == 0) base = reinterpret_cast<__nv_bfloat16 *>(e.q) + c;
        else if (!e.paged.slab) base = reinterpret_cast<__nv_bfloat16 *>(which == 1 ? e.k_lin : e.v_lin) + c;
        else { paged = true; base = reinterpret_cast<__nv_bfloat16 *>(e.paged.slab) + (size_t)(which - 1) * 64 * d + c; }
    }
    const int rr = lane >> 2, c8 = (lane & 3) * 8;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int r = it * 8 + rr;
        const int64_t m = m_base + r;
        if (m < M) {
            const uint4 t = *reinterpret_cast<const uint4 *>(pb + r * kPitchB + (lane & 3) * 16);
            __nv_bfloat16 *dst = paged ? base + rowoff[r] + c8 : base + m * pitch + c8;
            *reinterpret_cast<uint4 *>(dst) = t;
        }
    }
    __syncwarp();
}

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, int64_t M, int N, int K,
               Epilogue epi, int *err)
{
    constexpr int STAGES = Cfg<BN>::kStages, kStage = Cfg<BN>::kStage;
    constexpr uint32_t kTmemCols = Cfg<BN>::kTmemCols;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float *patches = reinterpret_cast<float *>(smem + STAGES * kStage);
    int64_t *rowoffs = reinterpret_cast<int64_t *>(smem + STAGES * kStage + kEpiWarps * kPatchBytes);
    GemmBars *bars = reinterpret_cast<GemmBars *>(smem + STAGES * kStage + kEpiWarps * kPatchBytes + kEpiWarps * 32 * 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kblocks = K / BK;
    const int n_tiles_n = N / BN;
    const int64_t n_tiles = ((M + BM - 1) / BM) * n_tiles_n;

    // set-up that touches nothing earlier kernels wrote; it may run while the previous kernel is still finishing
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&bars->full[s], 1); tc::mbar_init(&bars->empty[s], 1); }
        for (int s = 0; s < 2; ++s) { tc::mbar_init(&bars->acc_full[s], 1); tc::mbar_init(&bars->acc_empty[s], kEpiWarps); }
        tc::fence_mbar_init();
        tc::tma_prefetch_desc(&tmA);
        tc::tma_prefetch_desc(&tmB);
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

    if (!live) {
    } else if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                const int m0 = (int)(t / n_tiles_n) * BM, n0 = (int)(t % n_tiles_n) * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    ok = tc::mbar_wait(&bars->empty[s], ((it / STAGES) & 1) ^ 1, err);
                    if (!ok) break;
                    tc::mbar_expect_tx(&bars->full[s], kStage);
                    uint8_t *a = smem + s * kStage;
                    tc::tma_load_2d(a, &tmA, kb * BK, m0, &bars->full[s]);
                    tc::tma_load_2d(a + kABytes, &tmB, kb * BK, n0, &bars->full[s]);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (the whole warp walks the loop so that
        // addresses stay warp-uniform; one elected lane issues the tcgen05 instructions)
        {
            constexpr uint32_t idesc = tc::make_idesc(BM, BN, 0, 0);
            uint32_t it = 0, ti = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++ti) {
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
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)     // 32 bytes of K per instruction: descriptor start address + 2
                            tc::mma_ss(tmem_base + as * BN, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
                        tc::mma_commit(&bars->empty[s]);       // frees the stage when these MMAs have read it
                        if (kb == kblocks - 1) tc::mma_commit(&bars->acc_full[as]);
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
        float *patch = patches + ew * (kPatchBytes / 4);
        int64_t *rowoff = rowoffs + ew * 32;
        const bool scatter = epi.mode == EPI_QKV && epi.paged.slab != nullptr;
        uint32_t ti = 0;
        bool ok = true;
        for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++ti) {
            const int64_t m0 = (t / n_tiles_n) * BM;
            const int n0 = (int)(t % n_tiles_n) * BN;
            const uint32_t as = ti & 1;
            const int64_t m_base = m0 + quad * 32;
            const int64_t m = m_base + lane;
            // K / V rows of a pre-infer call go straight into the user's pages: offset of (page, K, slot) per row
            int last_slot = -1, page = 0;
            if (scatter && epi.col0 + n0 + half * kColsPerWarp + kColsPerWarp - 1 >= epi.d_model) {
                int64_t off = 0;
                if (m < M) {
                    const int u = find_user(epi.row_off, epi.n_users, (int)m);
                    const int tt = (int)m - epi.row_off[u];
                    page = epi.paged.pt[epi.seqs[u].pt_base + (tt >> 6)];
                    off = (int64_t)page_elem_offset(epi.paged, page, 0, tt & 63);
                    if (tt == epi.seqs[u].n_q - 1) last_slot = tt & 63;
                }
                rowoff[lane] = off;
                __syncwarp();
            }
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
                    if (lane == 0) tc::mbar_arrive(&bars->acc_empty[as]);      // this warp's part of the accumulator is in registers
                }
                float v[32];
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(cc == 0 ? r0[i] : r1[i]);
                    const int n = n0 + half * kColsPerWarp + pass * 64 + cc * 32;
                    epilogue_chunk(epi, m_base, M, n, N, v, lane, patch, rowoff);
                    if (last_slot >= 0 && last_slot < 63 && epi.col0 + n >= epi.d_model) {
                        // last prefix row of a user: clear the unused slots of its last page (they are masked, but must hold finite values)
                        const int col = epi.col0 + n, which = col / epi.d_model, c = col - which * epi.d_model;
                        __nv_bfloat16 *slab = reinterpret_cast<__nv_bfloat16 *>(epi.paged.slab);
                        const uint4 z = make_uint4(0, 0, 0, 0);
                        for (int s = last_slot + 1; s < 64; ++s) {
                            uint4 *zp = reinterpret_cast<uint4 *>(slab + page_elem_offset(epi.paged, page, which - 1, s) + c);
                            zp[0] = z; zp[1] = z; zp[2] = z; zp[3] = z;
                        }
                    }
                }
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

template <int BN>
static cudaError_t launch_bn(const CUtensorMap &tmA, const CUtensorMap &tmB, int64_t M, int N, int K, const Epilogue &epi, int *err,
                             cudaStream_t stream)
{
    static int n_sms = 0;
    if (n_sms == 0) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BN>::kSmemBytes);
        if (e != cudaSuccess) { n_sms = 0; return e; }
    }
    const int64_t tiles = ((M + BM - 1) / BM) * (N / BN);
    const unsigned grid = (unsigned)(tiles < n_sms ? tiles : n_sms);
    return launch_dependent(gemm_tc_kernel<BN>, dim3(grid), dim3(kThreads), (size_t)Cfg<BN>::kSmemBytes, stream, tmA, tmB, M, N, K, epi, err);
}

cudaError_t launch_gemm_tc(const CUtensorMap &tmA, const CUtensorMap &tmB, int64_t M, int N, int K, const Epilogue &epi,
                           int *err, cudaStream_t stream, int64_t *launches)
{
    if (M == 0 || N == 0) return cudaSuccess;
    *launches += 1;
    return gemm_tile_n(N, K) == 256 ? launch_bn<256>(tmA, tmB, M, N, K, epi, err, stream) : launch_bn<128>(tmA, tmB, M, N, K, epi, err, stream);
}

}  // namespace relaygr

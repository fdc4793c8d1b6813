// bf16 GEMM on the 5th-generation tensor cores: C[m, n] = sum_k A[m, k] W[n, k] with fp32
// accumulators in TMEM.  TMA stages 128 x 64 (A) and BN x 64 (W) tiles in shared memory with
// the 128-byte swizzle; one elected thread issues tcgen05.mma (M = 128, N = BN, K = 16 per
// instruction); four epilogue warps read the accumulators back with tcgen05.ld and apply
// bias / SiLU / residual / the Q-K-V split with the K/V page scatter.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2-5 = epilogue (TMEM lane quadrant = warp index % 4).
// One output tile per CTA; two CTAs fit per SM so one tile's epilogue overlaps the other's mainloop.
#include "kernels.cuh"
#include "tc_common.cuh"

namespace relaygr {

namespace {

constexpr int BM = 128, BK = 64, STAGES = 3;

template <int BN> struct GemmSmem {
    static constexpr int kABytes = BM * BK * 2;
    static constexpr int kBBytes = BN * BK * 2;
    static constexpr int kStage = kABytes + kBBytes;
    static constexpr int kTotal = STAGES * kStage + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int BN>
__device__ __forceinline__ void epilogue_chunk(const Epilogue &e, int64_t m, int n, int N, const uint32_t (&acc)[32], bool row_ok)
{
    if (!row_ok) return;
    float v[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(acc[i]);
    if (e.bias) {
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
            const float4 b = *reinterpret_cast<const float4 *>(e.bias + n + i);
            v[i] += b.x; v[i + 1] += b.y; v[i + 2] += b.z; v[i + 3] += b.w;
        }
    }
    if (e.mode == EPI_RESID) {
        const float4 *r = reinterpret_cast<const float4 *>(e.resid + m * N + n);
        float4 *o = reinterpret_cast<float4 *>(e.out_f32 + m * N + n);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float4 t = r[i];
            t.x += v[4 * i]; t.y += v[4 * i + 1]; t.z += v[4 * i + 2]; t.w += v[4 * i + 3];
            o[i] = t;
        }
        return;
    }
    if (e.mode == EPI_STORE && e.silu) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = v[i] / (1.f + __expf(-v[i]));
    }
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) pk[i] = tc::pack_bf16(v[2 * i], v[2 * i + 1]);
    __nv_bfloat16 *dst;
    if (e.mode == EPI_STORE) {
        dst = reinterpret_cast<__nv_bfloat16 *>(e.out) + m * N + n;
    } else {
        const int col = e.col0 + n, d = e.d_model;
        const int which = col / d, c = col - which * d;
        if (which == 0) {
            dst = reinterpret_cast<__nv_bfloat16 *>(e.q) + m * d + c;
        } else if (!e.paged.slab) {
            dst = reinterpret_cast<__nv_bfloat16 *>(which == 1 ? e.k_lin : e.v_lin) + m * d + c;
        } else {
            const int u = find_user(e.row_off, e.n_users, (int)m);
            const int t = (int)m - e.row_off[u];
            const int page = e.paged.pt[e.seqs[u].pt_base + (t >> 6)];
            __nv_bfloat16 *slab = reinterpret_cast<__nv_bfloat16 *>(e.paged.slab);
            dst = slab + page_elem_offset(e.paged, page, which - 1, t & 63) + c;
            if (t == e.seqs[u].n_q - 1) {      // last prefix row: clear the unused slots of its page
                const uint4 z = make_uint4(0, 0, 0, 0);
                for (int s = (t & 63) + 1; s < 64; ++s) {
                    uint4 *zp = reinterpret_cast<uint4 *>(slab + page_elem_offset(e.paged, page, which - 1, s) + c);
                    zp[0] = z; zp[1] = z; zp[2] = z; zp[3] = z;
                }
            }
        }
    }
    uint4 *o = reinterpret_cast<uint4 *>(dst);
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
}

template <int BN>
__global__ void __launch_bounds__(192)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, int64_t M, int N, int K,
               Epilogue epi, int *err)
{
    using S = GemmSmem<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + STAGES * S::kStage);
    uint64_t *empty = full + STAGES;
    uint64_t *acc_full = empty + STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t m0 = (int64_t)blockIdx.y * BM;
    const int n0 = blockIdx.x * BN;
    const int kblocks = K / BK;
    __shared__ int s_abort;
    if (threadIdx.x == 0) s_abort = *reinterpret_cast<volatile int *>(err);
    __syncthreads();
    if (s_abort != 0) return;                                    // an earlier CTA gave up: do not pile on

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        tc::mbar_init(acc_full, 1);
        tc::fence_mbar_init();
        tc::tma_prefetch_desc(&tmA);
        tc::tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tc::tmem_alloc(tmem_slot, BN);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < kblocks; ++kb) {
                const int s = kb % STAGES;
                if (!tc::mbar_wait(&empty[s], ((kb / STAGES) & 1) ^ 1, err)) break;
                tc::mbar_expect_tx(&full[s], S::kStage);
                uint8_t *a = smem + s * S::kStage;
                tc::tma_load_2d(a, &tmA, kb * BK, (int)m0, &full[s]);
                tc::tma_load_2d(a + S::kABytes, &tmB, kb * BK, n0, &full[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = tc::make_idesc(BM, BN, 0, 0);
            bool ok = true;
            for (int kb = 0; kb < kblocks && ok; ++kb) {
                const int s = kb % STAGES;
                ok = tc::mbar_wait(&full[s], (kb / STAGES) & 1, err);
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t a = tc::smem_u32(smem + s * S::kStage);
                const uint64_t adesc = tc::smem_desc_sw128(a), bdesc = tc::smem_desc_sw128(a + S::kABytes);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)     // 32 bytes of K per instruction: descriptor start address + 2
                    tc::mma_ss(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
                tc::mma_commit(&empty[s]);             // frees the stage when these MMAs have read it
            }
            tc::mma_commit(acc_full);
        }
    } else {
        const int quad = warp & 3;                     // TMEM lanes this warp may touch: 32*quad .. 32*quad+31
        const bool ok = __all_sync(0xffffffffu, tc::mbar_wait(acc_full, 0, err));
        tc::tc_fence_after();
        const int64_t m = m0 + quad * 32 + lane;
        if (ok) {
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t acc[32];
                tc::tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)c, acc);
                tc::tmem_ld_wait();
                epilogue_chunk<BN>(epi, m, n0 + c, N, acc, m < M);
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem_base, BN);
}

}  // namespace

cudaError_t launch_gemm_tc(const CUtensorMap &tmA, const CUtensorMap &tmB, int64_t M, int N, int K, const Epilogue &epi,
                           int *err, cudaStream_t stream, int64_t *launches)
{
    if (M == 0 || N == 0) return cudaSuccess;
    constexpr int BN = 128;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmSmem<BN>::kTotal);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    dim3 grid((unsigned)(N / BN), (unsigned)((M + BM - 1) / BM));
    gemm_tc_kernel<BN><<<grid, 192, GemmSmem<BN>::kTotal, stream>>>(tmA, tmB, M, N, K, epi, err);
    *launches += 1;
    return cudaGetLastError();
}

}  // namespace relaygr

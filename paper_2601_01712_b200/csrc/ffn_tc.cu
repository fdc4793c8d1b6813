// The feed-forward half of a block in ONE kernel for d_model = 256:
//     x <- x + W2 SiLU(W1 LN(x; g, b) + b1) + b2
// Nothing but x and the weights touches global memory: the normalised tile, the hidden activations and the output
// accumulator live in shared memory and TMEM.  A CTA owns 128 rows and walks the hidden dimension in chunks of 128:
//     S  = A W1c^T            A = LN(x) tile [128 x 256] bf16 in shared memory (written once by the CTA itself),
//                             W1c = 128 rows of W1 by TMA; fp32 S [128 x 128] in TMEM
//     H  = SiLU(S + b1c)      four warps, one row per thread, bf16 H back into TMEM (the A operand of the next MMA)
//     O += H W2c^T            W2c = 128 columns of W2 by TMA; fp32 O [128 x 256] in TMEM
// and after the last chunk O + b2 goes to x as a bulk fp32 add-reduction (as in gemm_tc.cu).  The structure is the
// one of the attention kernel (S -> P -> O) with the softmax replaced by a pointwise function, so no running state.
//
// Warp roles (320 threads): warp 0 = TMA producer of the weight stream (a 4-stage ring of 32 KB: half a W1 chunk or
// half a W2 chunk per stage, issued in the order the MMAs consume them), warp 1 = TMEM owner + MMA issuer, warps 2-9 =
// LayerNorm of the CTA's rows, then SiLU of every chunk, then the final store (two warps per TMEM quadrant, each with half
// of the columns).  TMEM (all 512 columns):
// O 0..255, S double-buffered 256..383 and 384..511; H(c) (bf16) overwrites S(c) once that is in registers: the warp that
// read columns 64 h .. 64 h + 63 of S(c) writes its 64 hidden units into the first 32 of those columns.  The MMA warp issues S(0), S(1), then per chunk O += H(c) W2c^T followed by S(c+2):
// the tensor pipe executes in issue order, so S(c+2) cannot overwrite the buffer before H(c) has been consumed, and the
// S MMAs of the next two chunks are always queued while the SiLU warps work.
#include "kernels.cuh"
#include "tc_common.cuh"

namespace relaygr {

namespace {

constexpr int kD = 256;                              // d_model this kernel is built for (O fills half of TMEM)
constexpr int kRows = 128, kChunk = 128, kMaxF = 2048;
constexpr int kEpiThreads = 256, kThreads = 64 + kEpiThreads;
constexpr int kABytes = kRows * kD * 2;              // 64 KB: four K blocks of [128 rows x 64] bf16, 128-byte swizzle
constexpr int kKBlock = kRows * 64 * 2;              // 16 KB
constexpr int kStageBytes = 32 * 1024, kStages = 4;
constexpr int kOffW = kABytes;
constexpr int kOffB1 = kOffW + kStages * kStageBytes;
constexpr int kOffB2 = kOffB1 + kMaxF * 4;
constexpr int kOffG = kOffB2 + kD * 4;               // LayerNorm gain and offset, out-proj bias (kProj): 3 x 256 floats
constexpr int kOffStat = kOffG + 3 * kD * 4;         // partial row statistics exchanged between the two warps of a row: 2 x 2 x 128 floats
constexpr int kOffBars = kOffStat + 2 * 2 * kRows * 4;
constexpr int kSmemBytes = kOffBars + 256 + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
constexpr uint32_t kTmemCols = 512, kColO = 0, kColS = 256;      // S buffer i at kColS + 128 i; H(c) in the first 64 columns of S(c)'s buffer

struct Bars {
    uint64_t a_ready;                                 // LN(x) tile is in shared memory (256 arrivals)
    uint64_t w_full[kStages], w_empty[kStages];
    uint64_t s_full[2];                               // S(c) complete in buffer c & 1
    uint64_t h_full[2];                               // H(c) in TMEM (256 arrivals)
    uint64_t o_full;
    uint64_t att_full, o1_full, x_full[4], x_done;    // kProj: attention tile landed / att Wo^T complete / x rows landed / x consumed
    uint32_t tmem_slot;
    int abort_flag;
};
static_assert(sizeof(Bars) <= 256, "barrier block");

__device__ __forceinline__ float silu(float z)
{
    const float h = 0.5f * z;
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(h));
    return fmaf(h, t, h);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ uint4 *patch_chunk(uint8_t *patch, int r, int j)
{
    return reinterpret_cast<uint4 *>(patch + r * 128 + ((j ^ (r & 7)) << 4));
}

// kProj: the output projection of the attention block runs first, in the same kernel: O starts as att Wo^T, LayerNorm is
// taken of x + O + bo (the block's mid-point, never written), and the feed-forward MMAs accumulate on top, so that the
// final add-reduction adds (att Wo^T + bo) + (feed-forward + b2) to x in one go.
template <bool kProj>
__global__ void __launch_bounds__(kThreads, 1)
ffn_fused_kernel(const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmX,
                 const __grid_constant__ CUtensorMap tmAtt, const __grid_constant__ CUtensorMap tmWo,
                 const float *__restrict__ x, const float *__restrict__ g, const float *__restrict__ b, const float *__restrict__ b1,
                 const float *__restrict__ b2, const float *__restrict__ bo, int64_t M, int F, float eps, int *err)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sA = smem, *sW = smem + kOffW;
    float *b1s = reinterpret_cast<float *>(smem + kOffB1), *b2s = reinterpret_cast<float *>(smem + kOffB2);
    float *gs = reinterpret_cast<float *>(smem + kOffG), *bs = gs + kD, *bos = bs + kD;
    float *stat = reinterpret_cast<float *>(smem + kOffStat);
    Bars *bars = reinterpret_cast<Bars *>(smem + kOffBars);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_chunks = F / kChunk;
    const int64_t m0 = (int64_t)blockIdx.x * kRows;

    // set-up that touches nothing earlier kernels wrote
    if (threadIdx.x == 0) {
        tc::mbar_init(&bars->a_ready, kEpiThreads);
        for (int s = 0; s < kStages; ++s) { tc::mbar_init(&bars->w_full[s], 1); tc::mbar_init(&bars->w_empty[s], 1); }
        for (int i = 0; i < 2; ++i) { tc::mbar_init(&bars->s_full[i], 1); tc::mbar_init(&bars->h_full[i], kEpiThreads); }
        tc::mbar_init(&bars->o_full, 1);
        tc::mbar_init(&bars->att_full, 1); tc::mbar_init(&bars->o1_full, 1); tc::mbar_init(&bars->x_done, kEpiThreads);
        for (int i = 0; i < 4; ++i) tc::mbar_init(&bars->x_full[i], 1);
        tc::fence_mbar_init();
        tc::tma_prefetch_desc(&tmW1); tc::tma_prefetch_desc(&tmW2); tc::tma_prefetch_desc(&tmX);
    }
    if (warp == 1) {
        tc::tmem_alloc(&bars->tmem_slot, kTmemCols);
        tc::tmem_relinquish();
    }
    if (warp >= 2) {                                  // the biases are parameters: not written by earlier kernels
        for (int i = threadIdx.x - 64; i < F; i += kEpiThreads) b1s[i] = b1 ? b1[i] : 0.f;
        for (int i = threadIdx.x - 64; i < kD; i += kEpiThreads) {
            b2s[i] = (b2 ? b2[i] : 0.f) + (kProj && bo ? bo[i] : 0.f);      // what the final add-reduction adds beside O
            if (kProj) { gs[i] = g[i]; bs[i] = b[i]; bos[i] = bo ? bo[i] : 0.f; }
        }
    }
    grid_launch_dependents();
    grid_dependency_wait();                           // from here on: data of earlier kernels
    if (threadIdx.x == 0) bars->abort_flag = *reinterpret_cast<volatile int *>(err);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const bool live = bars->abort_flag == 0;

    if (!live) {
    } else if (warp == 0) {
        // ---------------------------------------------------------------- weight stream, in the order of consumption:
        // W1(0), W1(1); then per chunk c: W2(c), W1(c+2)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            auto load = [&](bool second, int c, int half) {
                if (!ok) return;
                const int s = it % kStages;
                ok = tc::mbar_wait(&bars->w_empty[s], ((it / kStages) & 1) ^ 1, err);
                if (!ok) return;
                tc::mbar_expect_tx(&bars->w_full[s], kStageBytes);
                uint8_t *dst = sW + s * kStageBytes;
                if (!second) {                        // rows c*128 .. +127 of W1 [F, 256], K blocks 2*half and 2*half + 1
                    tc::tma_load_2d(dst, &tmW1, (2 * half) * 64, c * kChunk, &bars->w_full[s]);
                    tc::tma_load_2d(dst + kKBlock, &tmW1, (2 * half + 1) * 64, c * kChunk, &bars->w_full[s]);
                } else {                              // all 256 rows of W2 [256, F], 64 hidden columns
                    tc::tma_load_2d(dst, &tmW2, c * kChunk + half * 64, 0, &bars->w_full[s]);
                }
                ++it;
            };
            if (kProj) {
                // the attention tile (A of the projection) where the normalised tile will go, Wo through the ring, then - once
                // the projection MMAs have read both - this CTA's rows of x into the ring's memory as 32 x 32 fp32 patches
                tc::mbar_expect_tx(&bars->att_full, kABytes);
                for (int kb = 0; kb < 4; ++kb) tc::tma_load_2d(sA + kb * kKBlock, &tmAtt, kb * 64, (int)m0, &bars->att_full);
                for (int kb = 0; kb < 4 && ok; ++kb, ++it) {
                    const int s = it % kStages;
                    ok = tc::mbar_wait(&bars->w_empty[s], ((it / kStages) & 1) ^ 1, err);
                    if (!ok) break;
                    tc::mbar_expect_tx(&bars->w_full[s], kStageBytes);
                    tc::tma_load_2d(sW + s * kStageBytes, &tmWo, kb * 64, 0, &bars->w_full[s]);
                }
                if (ok) ok = tc::mbar_wait(&bars->o1_full, 0, err);
                for (int rg = 0; rg < 4 && ok; ++rg) {
                    tc::mbar_expect_tx(&bars->x_full[rg], kStageBytes);
                    for (int cg = 0; cg < 8; ++cg)
                        tc::tma_load_2d(sW + (rg * 8 + cg) * 4096, &tmX, cg * 32, (int)(m0 + rg * 32), &bars->x_full[rg]);
                }
                if (ok) ok = tc::mbar_wait(&bars->x_done, 0, err);          // the LayerNorm has taken x: the ring is free for weights
            }
            load(false, 0, 0); load(false, 0, 1);
            if (n_chunks > 1) { load(false, 1, 0); load(false, 1, 1); }
            for (int c = 0; c < n_chunks; ++c) {
                load(true, c, 0); load(true, c, 1);
                if (c + 2 < n_chunks) { load(false, c + 2, 0); load(false, c + 2, 1); }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (convergent warp, one elected lane issues)
        constexpr uint32_t idesc_s = tc::make_idesc(kRows, kChunk, 0, 0);      // A and W1 both K-major
        constexpr uint32_t idesc_o = tc::make_idesc(kRows, kD, 0, 0);          // H from TMEM, W2 K-major
        uint32_t it = 0;
        bool ok = true;
        const uint32_t a0 = tc::smem_u32(sA);
        if (kProj) {                                  // O = att Wo^T: four K blocks, M128 N256
            ok = tc::mbar_wait(&bars->att_full, 0, err);
            for (int kb = 0; kb < 4 && ok; ++kb, ++it) {
                const int s = it % kStages;
                ok = tc::mbar_wait(&bars->w_full[s], (it / kStages) & 1, err);
                if (!ok) break;
                tc::tc_fence_after();
                const uint64_t adesc = tc::smem_desc_sw128(a0 + kb * kKBlock), bdesc = tc::smem_desc_sw128(tc::smem_u32(sW + s * kStageBytes));
                if (tc::elect_one()) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) tc::mma_ss(tmem_base + kColO, adesc + 2 * k, bdesc + 2 * k, idesc_o, (kb | k) != 0);
                    tc::mma_commit(&bars->w_empty[s]);
                    if (kb == 3) tc::mma_commit(&bars->o1_full);
                }
                __syncwarp();
            }
        }
        if (ok) ok = tc::mbar_wait(&bars->a_ready, 0, err);
        tc::tc_fence_after();
        auto issue_s = [&](int c) {                   // S(c) = A W1c^T: two stages, each two K blocks of 64
            const uint32_t scol = kColS + (c & 1) * kChunk;
            for (int half = 0; half < 2 && ok; ++half, ++it) {
                const int s = it % kStages;
                ok = tc::mbar_wait(&bars->w_full[s], (it / kStages) & 1, err);
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t w = tc::smem_u32(sW + s * kStageBytes);
                if (tc::elect_one()) {
#pragma unroll
                    for (int kb = 0; kb < 2; ++kb) {
                        const uint64_t adesc = tc::smem_desc_sw128(a0 + (2 * half + kb) * kKBlock), bdesc = tc::smem_desc_sw128(w + kb * kKBlock);
#pragma unroll
                        for (int k = 0; k < 4; ++k) tc::mma_ss(tmem_base + scol, adesc + 2 * k, bdesc + 2 * k, idesc_s, (half | kb | k) != 0);
                    }
                    tc::mma_commit(&bars->w_empty[s]);
                    if (half == 1) tc::mma_commit(&bars->s_full[c & 1]);
                }
                __syncwarp();
            }
        };
        auto issue_o = [&](int c) {                   // O += H(c) W2c^T: two stages of 64 hidden columns each
            const uint32_t hcol = kColS + (c & 1) * kChunk;
            for (int half = 0; half < 2 && ok; ++half, ++it) {
                const int s = it % kStages;
                ok = tc::mbar_wait(&bars->w_full[s], (it / kStages) & 1, err);
                if (!ok) break;
                tc::tc_fence_after();
                const uint64_t bdesc = tc::smem_desc_sw128(tc::smem_u32(sW + s * kStageBytes));
                if (tc::elect_one()) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)      // 16 hidden units per instruction: 8 TMEM columns of H, 32 bytes of every W2 row
                        tc::mma_ts(tmem_base + kColO, tmem_base + hcol + half * 64 + k * 8, bdesc + 2 * k, idesc_o, kProj || (c | half | k) != 0);
                    tc::mma_commit(&bars->w_empty[s]);
                    if (half == 1 && c == n_chunks - 1) tc::mma_commit(&bars->o_full);
                }
                __syncwarp();
            }
        };
        if (ok) issue_s(0);
        if (ok && n_chunks > 1) issue_s(1);
        for (int c = 0; c < n_chunks && ok; ++c) {
            ok = tc::mbar_wait(&bars->h_full[c & 1], (c >> 1) & 1, err);      // H(c) is in TMEM (and S(c) in registers)
            if (!ok) break;
            tc::tc_fence_after();
            issue_o(c);
            if (ok && c + 2 < n_chunks) issue_s(c + 2);                        // into the buffer H(c) sits in: executes after the MMAs above
        }
    } else {
        // ---------------------------------------------------------------- LayerNorm, SiLU, final store: eight warps, two per TMEM
        // quadrant; of a chunk's 128 hidden columns (and of O's 256) warp (quad, ch) takes half ch
        const int ew = warp - 2, quad = warp & 3, ch = ew >> 2;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        bool ok = true;
        if (kProj) {
            // mid = x + att Wo^T + bo, one row per thread (the layout TMEM delivers), this warp's 128 columns of it in registers;
            // a = LN(mid) into the tile the attention rows came in.  The row statistics need both column halves: the two warps
            // of a row exchange partial sums through shared memory.
            const int rr = quad * 32 + lane;
            ok = __all_sync(0xffffffffu, tc::mbar_wait(&bars->o1_full, 0, err));
            if (ok) ok = __all_sync(0xffffffffu, tc::mbar_wait(&bars->x_full[quad], 0, err));
            tc::tc_fence_after();
            float xp[128];
            float psum = 0.f;
#pragma unroll
            for (int gi = 0; gi < 4; ++gi) {
                const int cc = ch * 128 + gi * 32;
                uint32_t r[32];
                tc::tmem_ld32(lane_addr + kColO + cc, r);
                tc::tmem_ld_wait();
                const uint8_t *patch = sW + (quad * 8 + ch * 4 + gi) * 4096;
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) {
                    const uint4 xv = *patch_chunk(const_cast<uint8_t *>(patch), lane, jj);
                    const float4 q = *reinterpret_cast<const float4 *>(bos + cc + 4 * jj);
                    xp[gi * 32 + 4 * jj] = __uint_as_float(r[4 * jj]) + __uint_as_float(xv.x) + q.x;
                    xp[gi * 32 + 4 * jj + 1] = __uint_as_float(r[4 * jj + 1]) + __uint_as_float(xv.y) + q.y;
                    xp[gi * 32 + 4 * jj + 2] = __uint_as_float(r[4 * jj + 2]) + __uint_as_float(xv.z) + q.z;
                    xp[gi * 32 + 4 * jj + 3] = __uint_as_float(r[4 * jj + 3]) + __uint_as_float(xv.w) + q.w;
                    psum += (xp[gi * 32 + 4 * jj] + xp[gi * 32 + 4 * jj + 1]) + (xp[gi * 32 + 4 * jj + 2] + xp[gi * 32 + 4 * jj + 3]);
                }
            }
            stat[ch * kRows + rr] = psum;
            asm volatile("bar.sync %0, 64;" ::"r"(1 + quad) : "memory");      // the two warps that share these 32 rows
            const float mean = (stat[rr] + stat[kRows + rr]) * (1.f / kD);
            float pvar = 0.f;
#pragma unroll
            for (int i = 0; i < 128; ++i) { const float dlt = xp[i] - mean; pvar = fmaf(dlt, dlt, pvar); }
            stat[(2 + ch) * kRows + rr] = pvar;
            asm volatile("bar.sync %0, 64;" ::"r"(1 + quad) : "memory");      // the two warps that share these 32 rows
            const float rstd = rsqrtf((stat[2 * kRows + rr] + stat[3 * kRows + rr]) * (1.f / kD) + eps);
#pragma unroll
            for (int q16 = 0; q16 < 16; ++q16) {
                const int c = ch * 128 + q16 * 8;
                const float4 ga = *reinterpret_cast<const float4 *>(gs + c), gb = *reinterpret_cast<const float4 *>(gs + c + 4);
                const float4 ba = *reinterpret_cast<const float4 *>(bs + c), bb2 = *reinterpret_cast<const float4 *>(bs + c + 4);
                const float *v = xp + q16 * 8;
                uint4 o;
                o.x = tc::pack_bf16((v[0] - mean) * rstd * ga.x + ba.x, (v[1] - mean) * rstd * ga.y + ba.y);
                o.y = tc::pack_bf16((v[2] - mean) * rstd * ga.z + ba.z, (v[3] - mean) * rstd * ga.w + ba.w);
                o.z = tc::pack_bf16((v[4] - mean) * rstd * gb.x + bb2.x, (v[5] - mean) * rstd * gb.y + bb2.y);
                o.w = tc::pack_bf16((v[6] - mean) * rstd * gb.z + bb2.z, (v[7] - mean) * rstd * gb.w + bb2.w);
                const int kb = c >> 6, j = (c & 63) >> 3;
                *reinterpret_cast<uint4 *>(sA + kb * kKBlock + rr * 128 + ((j ^ (rr & 7)) << 4)) = o;
            }
            tc::fence_proxy_async();                  // generic-proxy writes of the tile before the tensor core reads it
            tc::tc_fence_before();
            tc::mbar_arrive(&bars->x_done);
            tc::mbar_arrive(&bars->a_ready);
        } else {
            // a[r, :] = LN(x[r, :]) for 16 rows per warp, all their loads in flight at once: lane l holds columns 8l .. 8l+7,
            // i.e. the 16-byte chunk (l & 7) of K block (l >> 3), stored with the 128-byte swizzle the MMA descriptor expects
            const float4 g0 = *reinterpret_cast<const float4 *>(g + 8 * lane), g1 = *reinterpret_cast<const float4 *>(g + 8 * lane + 4);
            const float4 c0 = *reinterpret_cast<const float4 *>(b + 8 * lane), c1 = *reinterpret_cast<const float4 *>(b + 8 * lane + 4);
            uint8_t *dst_kb = sA + (lane >> 3) * kKBlock;
            const int j = lane & 7;
            float4 v0[16], v1[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int64_t row = m0 + ew * 16 + i;
                if (row < M) {
                    v0[i] = *reinterpret_cast<const float4 *>(x + row * kD + 8 * lane);
                    v1[i] = *reinterpret_cast<const float4 *>(x + row * kD + 8 * lane + 4);
                } else {
                    v0[i] = make_float4(0.f, 0.f, 0.f, 0.f); v1[i] = v0[i];
                }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float mean = warp_sum((v0[i].x + v0[i].y) + (v0[i].z + v0[i].w) + (v1[i].x + v1[i].y) + (v1[i].z + v1[i].w)) * (1.f / kD);
                const float d0 = v0[i].x - mean, d1 = v0[i].y - mean, d2 = v0[i].z - mean, d3 = v0[i].w - mean;
                const float d4 = v1[i].x - mean, d5 = v1[i].y - mean, d6 = v1[i].z - mean, d7 = v1[i].w - mean;
                const float var = warp_sum(d0 * d0 + d1 * d1 + d2 * d2 + d3 * d3 + d4 * d4 + d5 * d5 + d6 * d6 + d7 * d7) * (1.f / kD);
                const float rstd = rsqrtf(var + eps);
                uint4 o;
                o.x = tc::pack_bf16(d0 * rstd * g0.x + c0.x, d1 * rstd * g0.y + c0.y);
                o.y = tc::pack_bf16(d2 * rstd * g0.z + c0.z, d3 * rstd * g0.w + c0.w);
                o.z = tc::pack_bf16(d4 * rstd * g1.x + c1.x, d5 * rstd * g1.y + c1.y);
                o.w = tc::pack_bf16(d6 * rstd * g1.z + c1.z, d7 * rstd * g1.w + c1.w);
                const int rr = ew * 16 + i;
                *reinterpret_cast<uint4 *>(dst_kb + rr * 128 + ((j ^ (rr & 7)) << 4)) = o;
            }
            tc::fence_proxy_async();                  // generic-proxy writes of the tile before the tensor core reads it
            tc::mbar_arrive(&bars->a_ready);
        }
        for (int c = 0; c < n_chunks && ok; ++c) {
            const int hb = c & 1;
            const uint32_t scol = kColS + hb * kChunk + ch * 64;          // this warp's 64 columns of S(c)
            ok = __all_sync(0xffffffffu, tc::mbar_wait(&bars->s_full[hb], (c >> 1) & 1, err));
            if (!ok) break;
            tc::tc_fence_after();
            // the warp's 64 S values, then SiLU and the bf16 H into the first 32 of those same columns
            uint32_t r0[32], r1[32];
            tc::tmem_ld32(lane_addr + scol, r0);
            tc::tmem_ld32(lane_addr + scol + 32, r1);
            tc::tmem_ld_wait();
            const float4 *bb = reinterpret_cast<const float4 *>(b1s + c * kChunk + ch * 64);
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float4 q = bb[i];
                pk[2 * i] = tc::pack_bf16(silu(__uint_as_float(r0[4 * i]) + q.x), silu(__uint_as_float(r0[4 * i + 1]) + q.y));
                pk[2 * i + 1] = tc::pack_bf16(silu(__uint_as_float(r0[4 * i + 2]) + q.z), silu(__uint_as_float(r0[4 * i + 3]) + q.w));
            }
            tc::tmem_st16(lane_addr + scol, pk);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float4 q = bb[8 + i];
                pk[2 * i] = tc::pack_bf16(silu(__uint_as_float(r1[4 * i]) + q.x), silu(__uint_as_float(r1[4 * i + 1]) + q.y));
                pk[2 * i + 1] = tc::pack_bf16(silu(__uint_as_float(r1[4 * i + 2]) + q.z), silu(__uint_as_float(r1[4 * i + 3]) + q.w));
            }
            tc::tmem_st16(lane_addr + scol + 16, pk);
            tc::tmem_st_wait();
            tc::tc_fence_before();
            tc::mbar_arrive(&bars->h_full[hb]);
        }
        // ---- x += O + b2: fp32 patches of 32 rows x 32 columns handed to the TMA unit (the weight ring is idle by now)
        if (ok) ok = __all_sync(0xffffffffu, tc::mbar_wait(&bars->o_full, 0, err));
        tc::tc_fence_after();
        if (ok && m0 + quad * 32 < M) {
#pragma unroll 1
            for (int pass = 0; pass < 4; ++pass) {
                const int cc = ch * 128 + pass * 32;
                uint8_t *patch = sW + (ew * 4 + pass) * 4096;                  // a patch of its own for each of the warp's 4 passes
                uint32_t r[32];
                tc::tmem_ld32(lane_addr + kColO + cc, r);
                tc::tmem_ld_wait();
                const float4 *bb = reinterpret_cast<const float4 *>(b2s + cc);
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) {
                    const float4 q = bb[jj];
                    *patch_chunk(patch, lane, jj) = make_uint4(__float_as_uint(__uint_as_float(r[4 * jj]) + q.x), __float_as_uint(__uint_as_float(r[4 * jj + 1]) + q.y),
                                                               __float_as_uint(__uint_as_float(r[4 * jj + 2]) + q.z), __float_as_uint(__uint_as_float(r[4 * jj + 3]) + q.w));
                }
                tc::fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    tc::tma_reduce_add_2d(&tmX, patch, cc, (int)(m0 + quad * 32));
                    tc::bulk_commit();
                }
            }
        }
        if (lane == 0) tc::bulk_wait_read<0>();       // the patches have been read; the grid's completion covers the writes
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

bool ffn_fused_supported(int d_model, int d_ff) { return d_model == kD && d_ff % kChunk == 0 && d_ff >= kChunk && d_ff <= kMaxF; }

cudaError_t launch_ffn_fused(const CUtensorMap &tmW1, const CUtensorMap &tmW2, const CUtensorMap &tmX, const float *x, const float *g,
                             const float *b, const float *b1, const float *b2, const CUtensorMap *tmAtt, const CUtensorMap *tmWo,
                             const float *bo, int64_t M, int d_ff, float eps, int *err, cudaStream_t stream, int64_t *launches)
{
    if (M == 0) return cudaSuccess;
    static PerDeviceValue attr_set;
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (!attr_set.get(dev)) {
        cudaError_t e = cudaFuncSetAttribute(ffn_fused_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_fused_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set.set(dev, 1);
    }
    *launches += 1;
    const dim3 grid((unsigned)((M + kRows - 1) / kRows));
    if (tmAtt && tmWo)
        return launch_dependent(ffn_fused_kernel<true>, grid, dim3(kThreads), (size_t)kSmemBytes, stream, 1, tmW1, tmW2, tmX, *tmAtt, *tmWo, x, g,
                                b, b1, b2, bo, M, d_ff, eps, err);
    return launch_dependent(ffn_fused_kernel<false>, grid, dim3(kThreads), (size_t)kSmemBytes, stream, 1, tmW1, tmW2, tmX, tmX, tmX, x, g, b, b1,
                            b2, bo, M, d_ff, eps, err);
}

}  // namespace relaygr

// CUDA-core kernels: the memory-bound steps of both models (gather, LayerNorm, scoring
// head) and the GEMM / attention of the fp32 model, whose 1e-4 tolerance rules out TF32.
#include "kernels.cuh"

namespace relaygr {

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kMaxChunks = 8;      // a lane keeps up to 8 chunks of 4 values: d_model <= 1024

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16 *p)
{
    const uint2 u = *reinterpret_cast<const uint2 *>(p);
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&u.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&u.y);
    return make_float4(__low2float(a), __high2float(a), __low2float(b), __high2float(b));
}
__device__ __forceinline__ void store4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16 *p, float4 v)
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t *>(&a);
    u.y = *reinterpret_cast<uint32_t *>(&b);
    *reinterpret_cast<uint2 *>(p) = u;
}

__device__ __forceinline__ int row_token_id(const RowSource &src, int64_t row)
{
    const int u = find_user(src.row_off, src.n_users, (int)row);
    int i = (int)row - src.row_off[u];
#pragma unroll
    for (int s = 0; s < 3; ++s) {
        if (!src.ids[s]) continue;
        const int len = src.off[s][u + 1] - src.off[s][u];
        if (i < len) return src.ids[s][src.off[s][u] + i];
        i -= len;
    }
    return 0;
}

template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
gather_rows_kernel(const T *__restrict__ emb, int64_t vocab, int d, const int32_t *__restrict__ ids, int64_t n, T *__restrict__ out, int *err)
{
    const int64_t row = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= n) return;
    int64_t id = ids[row];
    if (id < 0 || id >= vocab) {
        // an id outside the table: recorded in the status word (when there is one), and a row that exists is read instead
        if (err && lane == 0) atomicCAS(err, (int)STATUS_OK, (int)STATUS_BAD_INDEX);
        id = id < 0 ? 0 : vocab - 1;
    }
    // 16-byte copies: d * sizeof(T) is a multiple of 16
    const int n16 = d * (int)sizeof(T) / 16;
    const uint4 *s = reinterpret_cast<const uint4 *>(emb + id * d);
    uint4 *o = reinterpret_cast<uint4 *>(out + row * d);
    for (int i = lane; i < n16; i += 32) o[i] = s[i];
}

// LayerNorm of ROWS rows a warp holds in registers (NC chunks of 128 columns, 4 values per lane and chunk; padding chunks
// hold zeros), biased variance, fp32 statistics; rows from n_rows on are skipped.
template <typename T, int NC, int ROWS>
__device__ __forceinline__ void ln_rows_store(const float4 (&v)[ROWS][NC], int d, int lane, int64_t row0, int64_t n_rows,
                                              const float *__restrict__ g, const float *__restrict__ b, float eps, T *__restrict__ a)
{
    float4 gg[NC], bb[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int i = (c * 32 + lane) * 4;
        if (i < d) { gg[c] = load4(g + i); bb[c] = load4(b + i); }
    }
    const float inv_d = 1.f / (float)d;
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        if (row0 + r >= n_rows) break;
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < NC; ++c) s += (v[r][c].x + v[r][c].y) + (v[r][c].z + v[r][c].w);
        const float mean = warp_sum(s) * inv_d;
        float q = 0.f;
#pragma unroll
        for (int c = 0; c < NC; ++c)
            if ((c * 32 + lane) * 4 < d) {
                const float a0 = v[r][c].x - mean, a1 = v[r][c].y - mean, a2 = v[r][c].z - mean, a3 = v[r][c].w - mean;
                q += a0 * a0 + a1 * a1 + a2 * a2 + a3 * a3;
            }
        const float rstd = rsqrtf(warp_sum(q) * inv_d + eps);
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int i = (c * 32 + lane) * 4;
            if (i < d) {
                float4 o;
                o.x = (v[r][c].x - mean) * rstd * gg[c].x + bb[c].x;
                o.y = (v[r][c].y - mean) * rstd * gg[c].y + bb[c].y;
                o.z = (v[r][c].z - mean) * rstd * gg[c].z + bb[c].z;
                o.w = (v[r][c].w - mean) * rstd * gg[c].w + bb[c].w;
                store4(a + (row0 + r) * d + i, o);
            }
        }
    }
}

// x[r, :] = emb[id(r), :] widened to fp32, a[r, :] = LN(x[r, :]).  A warp takes ROWS consecutive rows: lane r walks the
// look-up chain of row r (user of the row, segment, token id - dependent loads), so the ROWS chains run side by side, and
// all table rows are requested before any arithmetic: the table rows are scattered over HBM, and one row per warp kept
// too few bytes in flight.
template <typename T, int NC, int ROWS>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
gather_ln_kernel(const T *__restrict__ emb, int64_t vocab, int d, RowSource src, int64_t n_rows,
                 const float *__restrict__ g, const float *__restrict__ b, float eps, float *__restrict__ x, T *__restrict__ a, int *err)
{
    grid_launch_dependents();
    grid_dependency_wait();
    const int64_t row0 = ((int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5)) * ROWS;
    const int lane = threadIdx.x & 31;
    if (row0 >= n_rows) return;
    long long my_id = 0;
    if (lane < ROWS && row0 + lane < n_rows) {
        my_id = row_token_id(src, row0 + lane);
        if (my_id < 0 || my_id >= vocab) {
            // an id outside the table: recorded in the status word, and a row that exists is read instead
            if (err) atomicCAS(err, (int)STATUS_OK, (int)STATUS_BAD_INDEX);
            my_id = my_id < 0 ? 0 : vocab - 1;
        }
    }
    float4 v[ROWS][NC];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        const T *e = emb + __shfl_sync(0xffffffffu, my_id, r) * d;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int i = (c * 32 + lane) * 4;
            v[r][c] = (row0 + r < n_rows && i < d) ? load4(e + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
#pragma unroll
    for (int r = 0; r < ROWS; ++r)
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int i = (c * 32 + lane) * 4;
            if (row0 + r < n_rows && i < d) store4(x + (row0 + r) * d + i, v[r][c]);
        }
    ln_rows_store<T, NC, ROWS>(v, d, lane, row0, n_rows, g, b, eps, a);
}

// The candidate rows of every user, moved together: row i of x_c / a_c is the i-th candidate of the call (score order).
// seqs holds the COMPACT descriptors: self_row0 = row of the user's first candidate in the full-row buffers.
template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
compact_rows_kernel(const float *__restrict__ x, const T *__restrict__ a, const SeqDesc *__restrict__ seqs, int n_users,
                    const int32_t *__restrict__ score_off, int64_t n_total, int d, float *__restrict__ x_c, T *__restrict__ a_c)
{
    grid_launch_dependents();
    grid_dependency_wait();
    const int64_t i = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (i >= n_total) return;
    const int u = find_user(score_off, n_users, (int)i);
    const int64_t src = (int64_t)seqs[u].self_row0 + (i - score_off[u]);
    const uint4 *xs = reinterpret_cast<const uint4 *>(x + src * d);
    uint4 *xd = reinterpret_cast<uint4 *>(x_c + i * d);
    for (int j = lane; j < d / 4; j += 32) xd[j] = xs[j];
    const uint4 *as = reinterpret_cast<const uint4 *>(a + src * d);
    uint4 *ad = reinterpret_cast<uint4 *>(a_c + i * d);
    for (int j = lane; j < d * (int)sizeof(T) / 16; j += 32) ad[j] = as[j];
}

// a[r, :] = LN(x[r, :]).  A warp takes ROWS consecutive rows at once and issues all their loads before any
// arithmetic, so that enough bytes are in flight per SM to reach HBM / L2 bandwidth; NC = chunks of 128 columns.
template <typename T, int NC, int ROWS>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
layernorm_kernel(const float *__restrict__ x, int d, int64_t n_rows, const float *__restrict__ g, const float *__restrict__ b,
                 float eps, T *__restrict__ a)
{
    grid_launch_dependents();
    grid_dependency_wait();
    const int64_t row0 = ((int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5)) * ROWS;
    const int lane = threadIdx.x & 31;
    if (row0 >= n_rows) return;
    float4 v[ROWS][NC];
#pragma unroll
    for (int r = 0; r < ROWS; ++r)
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int i = (c * 32 + lane) * 4;
            v[r][c] = (row0 + r < n_rows && i < d) ? load4(x + (row0 + r) * d + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    ln_rows_store<T, NC, ROWS>(v, d, lane, row0, n_rows, g, b, eps, a);
}

// score[i] = w . LN(x[row(i), :]; g, b) + bias for the candidate rows.  As in the kernels above a warp takes ROWS
// consecutive candidates, lane r resolves candidate r's row (user look-up: dependent loads), and all rows are requested
// before any arithmetic.
template <int NC, int ROWS>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
score_kernel(const float *__restrict__ x, int d, const SeqDesc *__restrict__ seqs, int n_users, int64_t n_total,
             const int32_t *__restrict__ score_off, const float *__restrict__ g, const float *__restrict__ b, float eps,
             const float *__restrict__ w, const float *__restrict__ bias, float *__restrict__ scores)
{
    grid_launch_dependents();
    grid_dependency_wait();
    const int64_t idx0 = ((int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5)) * ROWS;
    const int lane = threadIdx.x & 31;
    if (idx0 >= n_total) return;
    long long my_row = 0;
    if (lane < ROWS && idx0 + lane < n_total) {
        const int idx = (int)(idx0 + lane);
        const int u = find_user(score_off, n_users, idx);
        my_row = (long long)seqs[u].score_row0 + (idx - score_off[u]);
    }
    float4 v[ROWS][NC];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        const float *xr = x + __shfl_sync(0xffffffffu, my_row, r) * d;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int i = (c * 32 + lane) * 4;
            v[r][c] = (idx0 + r < n_total && i < d) ? load4(xr + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    float4 gg[NC], bb[NC], ww[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int i = (c * 32 + lane) * 4;
        if (i < d) { gg[c] = load4(g + i); bb[c] = load4(b + i); ww[c] = load4(w + i); }
    }
    const float inv_d = 1.f / (float)d, bias0 = bias ? bias[0] : 0.f;
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        if (idx0 + r >= n_total) break;
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < NC; ++c) s += (v[r][c].x + v[r][c].y) + (v[r][c].z + v[r][c].w);
        const float mean = warp_sum(s) * inv_d;
        float q = 0.f;
#pragma unroll
        for (int c = 0; c < NC; ++c)
            if ((c * 32 + lane) * 4 < d) {
                const float a0 = v[r][c].x - mean, a1 = v[r][c].y - mean, a2 = v[r][c].z - mean, a3 = v[r][c].w - mean;
                q += a0 * a0 + a1 * a1 + a2 * a2 + a3 * a3;
            }
        const float rstd = rsqrtf(warp_sum(q) * inv_d + eps);
        float acc = 0.f;
#pragma unroll
        for (int c = 0; c < NC; ++c)
            if ((c * 32 + lane) * 4 < d)
                acc += ((v[r][c].x - mean) * rstd * gg[c].x + bb[c].x) * ww[c].x + ((v[r][c].y - mean) * rstd * gg[c].y + bb[c].y) * ww[c].y +
                       ((v[r][c].z - mean) * rstd * gg[c].z + bb[c].z) * ww[c].z + ((v[r][c].w - mean) * rstd * gg[c].w + bb[c].w) * ww[c].w;
        acc = warp_sum(acc);
        if (lane == 0) scores[idx0 + r] = acc + bias0;
    }
}

// ---- epilogue shared by the CUDA-core GEMM (one element at a time) ----------------------------------

template <typename T>
__device__ __forceinline__ void epilogue_store(const Epilogue &e, int64_t m, int n, int N, float acc)
{
    float v = acc + (e.bias ? e.bias[n] : 0.f);
    if (e.mode == EPI_STORE) {
        if (e.silu) v = v / (1.f + expf(-v));
        reinterpret_cast<T *>(e.out)[m * N + n] = Num<T>::from_f(v);
    } else if (e.mode == EPI_RESID) {
        e.out_f32[m * N + n] = e.resid[m * N + n] + v;
    } else {
        const int col = e.col0 + n, d = e.d_model;
        const int which = col / d, c = col - which * d;
        if (which == 0) { reinterpret_cast<T *>(e.q)[m * d + c] = Num<T>::from_f(v); return; }
        if (!e.paged.slab) {
            T *dst = reinterpret_cast<T *>(which == 1 ? e.k_lin : e.v_lin);
            dst[m * d + c] = Num<T>::from_f(v);
            return;
        }
        const int u = find_user(e.row_off, e.n_users, (int)m);
        const int t = (int)m - e.row_off[u];
        const int page = e.paged.pt[e.seqs[u].pt_base + (t >> 6)];
        T *slab = reinterpret_cast<T *>(e.paged.slab);
        slab[page_elem_offset(e.paged, page, which - 1, t & 63) + c] = Num<T>::from_f(v);
        if (t == e.seqs[u].n_q - 1)      // last row of the prefix: clear the unused slots of its page
            for (int s = (t & 63) + 1; s < 64; ++s) slab[page_elem_offset(e.paged, page, which - 1, s) + c] = Num<T>::from_f(0.f);
    }
}

// 64x64 tile, K step 16, 256 threads, 4x4 outputs per thread.
template <typename T>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T *__restrict__ A, const T *__restrict__ W, int64_t M, int N, int K, Epilogue epi)
{
    __shared__ float As[16][64 + 4];
    __shared__ float Ws[16][64 + 4];
    const int tid = threadIdx.x;
    const int64_t m0 = (int64_t)blockIdx.y * 64;
    const int n0 = blockIdx.x * 64;
    const int tr = tid / 16, tc = tid % 16;
    float acc[4][4] = {};
    const int lr = tid / 4, lk = (tid % 4) * 4;      // each thread loads 4 consecutive k of one row
    for (int k0 = 0; k0 < K; k0 += 16) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = k0 + lk + j;
            const int64_t am = m0 + lr;
            const int wn = n0 + lr;
            As[lk + j][lr] = (am < M && k < K) ? Num<T>::to_f(A[am * K + k]) : 0.f;
            Ws[lk + j][lr] = (wn < N && k < K) ? Num<T>::to_f(W[(int64_t)wn * K + k]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            float a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[k][tr * 4 + i]; w[i] = Ws[k][tc * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + tr * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tc * 4 + j;
            if (n < N) epilogue_store<T>(epi, m, n, N, acc[i][j]);
        }
    }
}

// ---- attention, one warp per (row, head); lanes split d_head ------------------------------------------

template <typename T, int DH>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
attention_simt_kernel(const T *__restrict__ q, const T *__restrict__ k_lin, const T *__restrict__ v_lin, PagedKV paged,
                      const SeqDesc *__restrict__ seqs, const int32_t *__restrict__ row_off, int n_users, int64_t n_rows,
                      int n_heads, int attn_kind, T *__restrict__ out)
{
    constexpr int PER = DH / 32;
    const int64_t wid = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (wid >= n_rows * n_heads) return;
    const int64_t row = wid / n_heads;
    const int h = (int)(wid - row * n_heads);
    const int d = n_heads * DH;
    const int u = find_user(row_off, n_users, (int)row);
    const SeqDesc sd = seqs[u];
    const int tpos = sd.q_pos0 + ((int)row - sd.q_row0);
    const bool is_cand = tpos >= sd.causal_end;
    const float scale = rsqrtf((float)DH);

    float qv[PER], o[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) { qv[i] = Num<T>::to_f(q[row * d + h * DH + lane * PER + i]) * scale; o[i] = 0.f; }
    float m = -INFINITY, l = 0.f;

    auto step = [&](const T *kp, const T *vp) {
        float dot = 0.f;
#pragma unroll
        for (int i = 0; i < PER; ++i) dot += qv[i] * Num<T>::to_f(kp[lane * PER + i]);
        dot = warp_sum(dot);
        if (attn_kind == ATTN_POINTWISE) {
            // pointwise aggregation: weight SiLU(logit), normalised by the number of visible keys (counted in l)
            const float p = dot / (1.f + expf(-dot));
            l += 1.f;
#pragma unroll
            for (int i = 0; i < PER; ++i) o[i] += p * Num<T>::to_f(vp[lane * PER + i]);
            return;
        }
        const float mn = fmaxf(m, dot);
        const float corr = expf(m - mn), p = expf(dot - mn);
        l = l * corr + p;
#pragma unroll
        for (int i = 0; i < PER; ++i) o[i] = o[i] * corr + p * Num<T>::to_f(vp[lane * PER + i]);
        m = mn;
    };

    // paged keys: positions 0 .. n_paged-1
    const int lim = is_cand ? sd.causal_end : tpos + 1;     // keys at positions < lim are visible
    const int np = min(sd.n_paged, lim);
    const T *slab = reinterpret_cast<const T *>(paged.slab);
    for (int j = 0; j < np; ++j) {
        const int page = paged.pt[sd.pt_base + (j >> 6)];
        step(slab + page_elem_offset(paged, page, 0, j & 63) + h * DH, slab + page_elem_offset(paged, page, 1, j & 63) + h * DH);
    }
    // linear keys: positions lin_pos0 .. lin_pos0+n_lin-1
    const int nl = min(sd.n_lin, lim - sd.lin_pos0);
    for (int j = 0; j < nl; ++j) {
        const int64_t r = sd.lin_row0 + j;
        step(k_lin + r * d + h * DH, v_lin + r * d + h * DH);
    }
    // a candidate also sees itself
    if (is_cand) step(k_lin + row * d + h * DH, v_lin + row * d + h * DH);

    const float inv = 1.f / l;
#pragma unroll
    for (int i = 0; i < PER; ++i) out[row * d + h * DH + lane * PER + i] = Num<T>::from_f(o[i] * inv);
}

inline unsigned blocks_for(int64_t warps) { return (unsigned)((warps + kWarpsPerBlock - 1) / kWarpsPerBlock); }

}  // namespace

template <typename T>
cudaError_t launch_gather_rows(const T *emb, int64_t vocab, int d, const int32_t *ids, int64_t n, T *out, int *err,
                               cudaStream_t stream, int64_t *launches)
{
    if (n == 0) return cudaSuccess;
    gather_rows_kernel<T><<<blocks_for(n), kWarpsPerBlock * 32, 0, stream>>>(emb, vocab, d, ids, n, out, err);
    *launches += 1;
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_gather_ln(const T *emb, int64_t vocab, int d, RowSource src, int64_t n_rows, const float *g,
                             const float *b, float eps, float *x, T *a, int *err, cudaStream_t stream, int64_t *launches)
{
    if (n_rows == 0) return cudaSuccess;
    const int nc = (d + 127) / 128;
    cudaError_t e;
#define RELAYGR_GLN(NC, ROWS)                                                                                             \
    e = launch_dependent(gather_ln_kernel<T, NC, ROWS>, dim3(blocks_for((n_rows + ROWS - 1) / ROWS)), dim3(kWarpsPerBlock * 32), 0, stream, 1, \
                         emb, vocab, d, src, n_rows, g, b, eps, x, a, err)
    if (nc <= 1) RELAYGR_GLN(1, 4);
    else if (nc <= 2) RELAYGR_GLN(2, 4);
    else if (nc <= 4) RELAYGR_GLN(4, 4);
    else RELAYGR_GLN(8, 1);
#undef RELAYGR_GLN
    *launches += 1;
    return e;
}

template <typename T>
cudaError_t launch_layernorm(const float *x, int d, int64_t n_rows, const float *g, const float *b, float eps, T *a,
                             cudaStream_t stream, int64_t *launches)
{
    if (n_rows == 0) return cudaSuccess;
    const int nc = (d + 127) / 128;
    cudaError_t e;
#define RELAYGR_LN(NC, ROWS)                                                                                              \
    e = launch_dependent(layernorm_kernel<T, NC, ROWS>, dim3(blocks_for((n_rows + ROWS - 1) / ROWS)), dim3(kWarpsPerBlock * 32), 0, stream, 1, \
                         x, d, n_rows, g, b, eps, a)
    if (nc <= 1) RELAYGR_LN(1, 4);
    else if (nc <= 2) RELAYGR_LN(2, 4);
    else if (nc <= 4) RELAYGR_LN(4, 4);
    else RELAYGR_LN(8, 1);
#undef RELAYGR_LN
    *launches += 1;
    return e;
}

cudaError_t launch_score(const float *x, int d, const SeqDesc *seqs, int n_users, int64_t n_total, const int32_t *score_off,
                         const float *g, const float *b, float eps, const float *w, const float *bias, float *scores,
                         cudaStream_t stream, int64_t *launches)
{
    if (n_total == 0) return cudaSuccess;
    const int nc = (d + 127) / 128;
    cudaError_t e;
#define RELAYGR_SCORE(NC, ROWS)                                                                                           \
    e = launch_dependent(score_kernel<NC, ROWS>, dim3(blocks_for((n_total + ROWS - 1) / ROWS)), dim3(kWarpsPerBlock * 32), 0, stream, 1, x, d, \
                         seqs, n_users, n_total, score_off, g, b, eps, w, bias, scores)
    if (nc <= 1) RELAYGR_SCORE(1, 4);
    else if (nc <= 2) RELAYGR_SCORE(2, 4);
    else if (nc <= 4) RELAYGR_SCORE(4, 2);
    else RELAYGR_SCORE(8, 1);
#undef RELAYGR_SCORE
    *launches += 1;
    return e;
}

template <typename T>
cudaError_t launch_compact_rows(const float *x, const T *a, const SeqDesc *seqs, int n_users, const int32_t *score_off, int64_t n_total,
                                int d, float *x_c, T *a_c, cudaStream_t stream, int64_t *launches)
{
    if (n_total == 0) return cudaSuccess;
    *launches += 1;
    return launch_dependent(compact_rows_kernel<T>, dim3(blocks_for(n_total)), dim3(kWarpsPerBlock * 32), 0, stream, 1, x, a, seqs, n_users,
                            score_off, n_total, d, x_c, a_c);
}

template <typename T>
cudaError_t launch_gemm_simt(const T *A, const T *W, int64_t M, int N, int K, const Epilogue &epi, cudaStream_t stream,
                             int64_t *launches)
{
    if (M == 0 || N == 0) return cudaSuccess;
    dim3 grid((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64));
    gemm_simt_kernel<T><<<grid, 256, 0, stream>>>(A, W, M, N, K, epi);
    *launches += 1;
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_attention_simt(const T *q, const T *k_lin, const T *v_lin, PagedKV paged, const SeqDesc *seqs,
                                  const int32_t *row_off, int n_users, int64_t n_rows, int n_heads, int d_head, int attn_kind,
                                  T *out, cudaStream_t stream, int64_t *launches)
{
    if (n_rows == 0) return cudaSuccess;
    const unsigned blocks = blocks_for(n_rows * n_heads);
    if (d_head == 32)
        attention_simt_kernel<T, 32><<<blocks, kWarpsPerBlock * 32, 0, stream>>>(q, k_lin, v_lin, paged, seqs, row_off, n_users,
                                                                                 n_rows, n_heads, attn_kind, out);
    else if (d_head == 64)
        attention_simt_kernel<T, 64><<<blocks, kWarpsPerBlock * 32, 0, stream>>>(q, k_lin, v_lin, paged, seqs, row_off, n_users,
                                                                                 n_rows, n_heads, attn_kind, out);
    else
        return cudaErrorInvalidValue;
    *launches += 1;
    return cudaGetLastError();
}

#define RELAYGR_INSTANTIATE(T)                                                                                              \
    template cudaError_t launch_gather_rows<T>(const T *, int64_t, int, const int32_t *, int64_t, T *, int *, cudaStream_t, int64_t *); \
    template cudaError_t launch_gather_ln<T>(const T *, int64_t, int, RowSource, int64_t, const float *, const float *, float,  \
                                             float *, T *, int *, cudaStream_t, int64_t *);                                 \
    template cudaError_t launch_layernorm<T>(const float *, int, int64_t, const float *, const float *, float, T *,          \
                                             cudaStream_t, int64_t *);                                                      \
    template cudaError_t launch_compact_rows<T>(const float *, const T *, const SeqDesc *, int, const int32_t *, int64_t, int, \
                                                float *, T *, cudaStream_t, int64_t *);                                     \
    template cudaError_t launch_gemm_simt<T>(const T *, const T *, int64_t, int, int, const Epilogue &, cudaStream_t,        \
                                             int64_t *);                                                                    \
    template cudaError_t launch_attention_simt<T>(const T *, const T *, const T *, PagedKV, const SeqDesc *, const int32_t *, \
                                                  int, int64_t, int, int, int, T *, cudaStream_t, int64_t *);
RELAYGR_INSTANTIATE(float)
RELAYGR_INSTANTIATE(__nv_bfloat16)

}  // namespace relaygr

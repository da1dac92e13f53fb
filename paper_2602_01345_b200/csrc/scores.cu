// Alternative per-token selection scores of the paper's selection-metric ablation (the table that
// compares entropy with an attention-based and an MSE-based criterion). Either score feeds the same
// nova_select_topk as the entropy does. These are comparison criteria, not the method's hot path:
// the kernels are straightforward (warp-per-row for the MSE score; warp-level matrix fragments for
// the attention mass) and are not tuned beyond that.
#include "common.cuh"

#include <mma.h>

namespace {

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ void unpack2(uint32_t w, float& lo, float& hi)
{
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xffff0000u);
}

// ---- MSE score: mean over channels of (x - bilinear resize of the previous scale's map)^2 -----------
constexpr int kMseWarps = 8;

__global__ void __launch_bounds__(kMseWarps * 32)
score_mse_kernel(const uint4* __restrict__ x, const uint4* __restrict__ ref, int B, int hp, int wp, int h, int w,
                 int vec_per_row, float* __restrict__ score)
{
    const int lane = threadIdx.x & 31;
    const long r = (long)blockIdx.x * kMseWarps + (threadIdx.x >> 5);
    const int N = h * w;
    if (r >= (long)B * N) return;
    const int b = (int)(r / N), i = (int)(r - (long)b * N);
    const int oy = i / w, ox = i - oy * w;
    float sy = ((float)oy + 0.5f) * ((float)hp / (float)h) - 0.5f;
    float sx = ((float)ox + 0.5f) * ((float)wp / (float)w) - 0.5f;
    sy = fmaxf(sy, 0.f);
    sx = fmaxf(sx, 0.f);
    const int y0 = min((int)sy, hp - 1), x0 = min((int)sx, wp - 1);
    const int y1 = min(y0 + 1, hp - 1), x1 = min(x0 + 1, wp - 1);
    const float fy = sy - (float)y0, fx = sx - (float)x0;
    const float w00 = (1.f - fy) * (1.f - fx), w01 = (1.f - fy) * fx, w10 = fy * (1.f - fx), w11 = fy * fx;
    const uint4* c00 = ref + (((long)b * hp + y0) * wp + x0) * vec_per_row;
    const uint4* c01 = ref + (((long)b * hp + y0) * wp + x1) * vec_per_row;
    const uint4* c10 = ref + (((long)b * hp + y1) * wp + x0) * vec_per_row;
    const uint4* c11 = ref + (((long)b * hp + y1) * wp + x1) * vec_per_row;
    const uint4* xr = x + r * vec_per_row;
    float acc = 0.f;
    for (int v = lane; v < vec_per_row; v += 32) {
        const uint4 xv = xr[v], a = c00[v], bq = c01[v], c = c10[v], d = c11[v];
        const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {bq.x, bq.y, bq.z, bq.w};
        const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, dw[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float xl, xh, al, ah, bl, bh, cl, ch, dl, dh;
            unpack2(xw[q], xl, xh);
            unpack2(aw[q], al, ah);
            unpack2(bw[q], bl, bh);
            unpack2(cw[q], cl, ch);
            unpack2(dw[q], dl, dh);
            const float d0 = xl - (w00 * al + w01 * bl + w10 * cl + w11 * dl);
            const float d1 = xh - (w00 * ah + w01 * bh + w10 * ch + w11 * dh);
            acc = fmaf(d0, d0, acc);
            acc = fmaf(d1, d1, acc);
        }
    }
    acc = warp_sum(acc);
    if (lane == 0) score[r] = acc / (float)(vec_per_row * 8);
}

// ---- attention mass ------------------------------------------------------------------------------
// Two passes over S = q K^T / sqrt(dh) per (image, head), S tiles of 64 queries x 64 keys on
// warp-level matrix fragments (bf16 in, fp32 out), one warp per 16 query rows:
//   pass 1  row statistics: lse[b, h, q] = log2-domain log-sum-exp of row q over all keys
//   pass 2  column sums over the scale's own keys: one CTA per 64 keys walks all heads and query
//           tiles in a fixed order (deterministic, no atomics) and adds up 2^(s - lse).
constexpr int kAmTile = 64;
constexpr int kAmThreads = 128;

template <int DH>
struct AmSmem {
    __nv_bfloat16 q[kAmTile][DH + 8];      // +8: rows 16 bytes apart in bank phase
    __nv_bfloat16 k[kAmTile][DH + 8];
    float s[4][16][kAmTile + 4];
};

// S tile of this warp's 16 query rows against the 64 keys in sm.k, into sm.s[warp]
template <int DH>
__device__ __forceinline__ void am_scores(AmSmem<DH>& sm, int warp)
{
    using namespace nvcuda;
    wmma::fragment<wmma::accumulator, 16, 16, 16, float> acc[4];
#pragma unroll
    for (int n = 0; n < 4; ++n) wmma::fill_fragment(acc[n], 0.f);
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
        wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> a;
        wmma::load_matrix_sync(a, &sm.q[warp * 16][kk * 16], DH + 8);
#pragma unroll
        for (int n = 0; n < 4; ++n) {
            wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::col_major> bfr;
            wmma::load_matrix_sync(bfr, &sm.k[n * 16][kk * 16], DH + 8);
            wmma::mma_sync(acc[n], a, bfr, acc[n]);
        }
    }
#pragma unroll
    for (int n = 0; n < 4; ++n) wmma::store_matrix_sync(&sm.s[warp][0][n * 16], acc[n], kAmTile + 4, wmma::mem_row_major);
    __syncwarp();
}

// loads rows [row0, row0 + 64) x channels [c0, c0 + DH) of a [rows_total, C] bf16 matrix (zero past the end)
template <int DH>
__device__ __forceinline__ void am_load_tile(__nv_bfloat16 (*dst)[DH + 8], const __nv_bfloat16* src, long row0, long rows_total,
                                             int C, int c0)
{
    constexpr int kVec = DH / 8;
    for (int i = threadIdx.x; i < kAmTile * kVec; i += kAmThreads) {
        const int r = i / kVec, v = i - r * kVec;
        uint4 val = make_uint4(0, 0, 0, 0);
        if (row0 + r < rows_total) val = *(const uint4*)(src + (row0 + r) * C + c0 + v * 8);
        *(uint4*)&dst[r][v * 8] = val;
    }
}

template <int DH>
__global__ void __launch_bounds__(kAmThreads)
attn_mass_rows(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
               const __nv_bfloat16* __restrict__ k_cache, const int32_t* __restrict__ kv_len,
               int N, int C, int Lmax, float scale_log2e, float* __restrict__ lse)
{
    extern __shared__ __align__(128) uint8_t am_raw[];
    AmSmem<DH>& sm = *reinterpret_cast<AmSmem<DH>*>(am_raw);
    const int b = blockIdx.z, hd = blockIdx.y, q0 = blockIdx.x * kAmTile, n_heads = gridDim.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_old = kv_len ? min(max(kv_len[b], 0), Lmax) : 0;
    const int n_keys = n_old + N;
    am_load_tile<DH>(sm.q, q + (long)b * N * C, q0, N, C, hd * DH);
    // every lane pair owns one row of the warp's 16: lane = 2 * row + half, 32 columns each
    const int row = lane >> 1, half = lane & 1;
    float m = -INFINITY, l = 0.f;
    for (int j0 = 0; j0 < n_keys; j0 += kAmTile) {
        __syncthreads();        // the previous tile's readers are done with sm.k
        // a key tile may straddle the cache / own-keys boundary: row by row
        constexpr int kVec = DH / 8;
        for (int i = threadIdx.x; i < kAmTile * kVec; i += kAmThreads) {
            const int r = i / kVec, v = i - r * kVec;
            const int j = j0 + r;
            uint4 val = make_uint4(0, 0, 0, 0);
            if (j < n_old) val = *(const uint4*)(k_cache + ((long)b * Lmax + j) * C + hd * DH + v * 8);
            else if (j < n_keys) val = *(const uint4*)(k + ((long)b * N + (j - n_old)) * C + hd * DH + v * 8);
            *(uint4*)&sm.k[r][v * 8] = val;
        }
        __syncthreads();
        am_scores<DH>(sm, warp);
        const int valid = min(kAmTile, n_keys - j0);
        float tm = -INFINITY;
        for (int c = half * 32; c < half * 32 + 32; ++c)
            if (c < valid) tm = fmaxf(tm, sm.s[warp][row][c] * scale_log2e);
        tm = fmaxf(tm, __shfl_xor_sync(0xffffffffu, tm, 1));
        const float m_new = fmaxf(m, tm);
        float part = 0.f;
        for (int c = half * 32; c < half * 32 + 32; ++c)
            if (c < valid) part += exp2f(sm.s[warp][row][c] * scale_log2e - m_new);
        part += __shfl_xor_sync(0xffffffffu, part, 1);
        l = l * exp2f(m - m_new) + part;      // exp2f(-inf) = 0 on the first tile
        m = m_new;
        __syncwarp();
    }
    const int qi = q0 + warp * 16 + row;
    if (half == 0 && qi < N) lse[((long)b * n_heads + hd) * N + qi] = m + log2f(l);
}

template <int DH>
__global__ void __launch_bounds__(kAmThreads)
attn_mass_cols(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
               int N, int C, int n_heads, float scale_log2e, const float* __restrict__ lse, float* __restrict__ score)
{
    extern __shared__ __align__(128) uint8_t am_raw[];
    AmSmem<DH>& sm = *reinterpret_cast<AmSmem<DH>*>(am_raw);
    __shared__ float colsum[4][kAmTile];
    const int b = blockIdx.y, j0 = blockIdx.x * kAmTile;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float acc0 = 0.f, acc1 = 0.f;      // this lane's two key columns (lane, lane + 32), summed over the warp's rows
    for (int hd = 0; hd < n_heads; ++hd) {
        __syncthreads();
        am_load_tile<DH>(sm.k, k + (long)b * N * C, j0, N, C, hd * DH);
        for (int q0 = 0; q0 < N; q0 += kAmTile) {
            __syncthreads();
            am_load_tile<DH>(sm.q, q + (long)b * N * C, q0, N, C, hd * DH);
            __syncthreads();
            am_scores<DH>(sm, warp);
            const float* lrow = lse + ((long)b * n_heads + hd) * N;
            for (int r = 0; r < 16; ++r) {
                const int qi = q0 + warp * 16 + r;
                if (qi >= N) break;
                const float e = lrow[qi];
                acc0 += exp2f(sm.s[warp][r][lane] * scale_log2e - e);
                acc1 += exp2f(sm.s[warp][r][lane + 32] * scale_log2e - e);
            }
            __syncwarp();
        }
    }
    colsum[warp][lane] = acc0;
    colsum[warp][lane + 32] = acc1;
    __syncthreads();
    if (threadIdx.x < kAmTile) {
        const int j = j0 + threadIdx.x;
        if (j < N) {
            const float tot = (colsum[0][threadIdx.x] + colsum[1][threadIdx.x]) + (colsum[2][threadIdx.x] + colsum[3][threadIdx.x]);
            score[(long)b * N + j] = tot / ((float)n_heads * (float)N);
        }
    }
}

template <int DH>
nova_status launch_mass(nova_ctx* ctx, const void* q, const void* k, const void* k_cache, const int32_t* kv_len,
                        int B, int N, int C, int n_heads, int Lmax, float* lse, float* score, cudaStream_t st)
{
    const int smem = (int)sizeof(AmSmem<DH>);
    static bool attr_done[64];
    if (ctx->device < 64 && !attr_done[ctx->device]) {
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(attn_mass_rows<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(attn_mass_cols<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr_done[ctx->device] = true;
    }
    const float scale_log2e = (float)((1.0 / sqrt((double)DH)) * 1.4426950408889634);
    const int tiles = (N + kAmTile - 1) / kAmTile;
    typedef const __nv_bfloat16* cbf;
    {
        nova_launch_scope scope(ctx, NOVA_K_SCORE, st);
        attn_mass_rows<DH><<<dim3(tiles, n_heads, B), kAmThreads, smem, st>>>((cbf)q, (cbf)k, (cbf)k_cache, kv_len, N, C, Lmax,
                                                                             scale_log2e, lse);
    }
    {
        nova_launch_scope scope(ctx, NOVA_K_SCORE, st);
        attn_mass_cols<DH><<<dim3(tiles, B), kAmThreads, smem, st>>>((cbf)q, (cbf)k, N, C, n_heads, scale_log2e, lse, score);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

}  // namespace

extern "C" nova_status nova_score_mse(nova_ctx* ctx, const void* x, const void* ref_prev, int B, int hp, int wp,
                                      int h, int w, int C, float* score, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (B < 0 || h < 0 || w < 0 || C < 1) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_score_mse: bad sizes");
    const long total = (long)B * h * w;
    if (total == 0) return NOVA_OK;
    if (total > 0x7fffffffL) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_score_mse: too many tokens");
    if (C % 8) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_score_mse: C must be a multiple of 8");
    if (!x || !ref_prev || !score || hp < 1 || wp < 1) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_score_mse: null pointer or empty reference map");
    if (!nova_aligned16(x) || !nova_aligned16(ref_prev)) return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_score_mse: tensors must be 16-byte aligned");
    NOVA_DEVICE_GUARD(ctx, "nova_score_mse");
    const unsigned blocks = (unsigned)((total + kMseWarps - 1) / kMseWarps);
    nova_launch_scope scope(ctx, NOVA_K_SCORE, (cudaStream_t)stream);
    score_mse_kernel<<<blocks, kMseWarps * 32, 0, (cudaStream_t)stream>>>((const uint4*)x, (const uint4*)ref_prev, B, hp, wp, h, w,
                                                                         C / 8, score);
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

extern "C" nova_status nova_score_attention_mass(nova_ctx* ctx, const void* q, const void* k, const void* k_cache,
                                                 const int32_t* kv_len, int B, int N, int C, int n_heads, int Lmax,
                                                 float* lse_scratch, float* score, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (B < 0 || N < 0 || C < 1 || n_heads < 1 || Lmax < 0) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_score_attention_mass: bad sizes");
    if ((long)B * N == 0) return NOVA_OK;
    if (C % n_heads || (C / n_heads != 64 && C / n_heads != 128))
        return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_score_attention_mass: head size must be 64 or 128");
    if (B > 65535 || n_heads > 65535) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_score_attention_mass: too many images or heads");
    if (!q || !k || !score || !lse_scratch || (kv_len && !k_cache))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_score_attention_mass: null pointer");
    if (!nova_aligned16(q) || !nova_aligned16(k) || !nova_aligned16(k_cache))
        return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_score_attention_mass: tensors must be 16-byte aligned");
    NOVA_DEVICE_GUARD(ctx, "nova_score_attention_mass");
    cudaStream_t st = (cudaStream_t)stream;
    if (C / n_heads == 64) return launch_mass<64>(ctx, q, k, k_cache, kv_len, B, N, C, n_heads, Lmax, lse_scratch, score, st);
    return launch_mass<128>(ctx, q, k, k_cache, kv_len, B, N, C, n_heads, Lmax, lse_scratch, score, st);
}

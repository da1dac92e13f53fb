// Eq. 14 on the kept tokens: gather + LayerNorm, QKV projection with K/V cache append,
// attention, output projection + residual, LayerNorm, MLP with tanh-GELU + residual.
// This file holds the small memory-bound kernels (row maps, LayerNorm, kv_len update), the
// workspace layout and the launch sequence; the contractions live in gemm.cu / attention.cu.
#include "common.cuh"

namespace {

// ---- row maps ---------------------------------------------------------------------------
// src_row[r] = b*N + keep_idx[r]            row of x_in feeding compacted row r
// kv_row[r]  = b*Lmax + kv_len[b] + (r - cu_keep[b])   cache row receiving r's k and v
//              (-1 and a SHAPE flag if the image's cache would overflow)
// Both are produced by the first LayerNorm (one warp per compacted row) on its way: it needs
// src_row to gather its input anyway.
struct RowMapArgs {
    const int32_t* keep_idx;
    const int32_t* cu_keep;
    const int32_t* kv_len;
    int B, N, Lmax;
    int32_t* src_row;
    int32_t* kv_row;
    int32_t* img_row;     // image of compacted row r
    unsigned int* status;
};

// Per-image modulation of a LayerNorm's output (adaptive LayerNorm): out * (1 + scale[b]) + shift[b].
// scale / shift: [B, C] bf16 or NULL; img_row gives b for the kernels that do not build the maps.
struct LnModArgs {
    const uint4* scale;
    const uint4* shift;
    const int32_t* img_row;
};

// ---- LayerNorm ----------------------------------------------------------------------------
// One warp per row; the row (C <= 32*8*VEC bf16) stays in registers between the mean, the
// variance and the normalisation, so x is read once and out written once.
constexpr int kLnWarps = 8;

__device__ __forceinline__ uint4 ld_nc_stream(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Three resident blocks per SM (80 registers): with two (94 registers) a launch of 1024 blocks ran 3.5
// waves of load-then-compute and sat at 0.41 of the HBM peak.
template <int VEC, bool MAPS, bool MOD>
__global__ void __launch_bounds__(kLnWarps * 32, 3)
layernorm_rows(const uint4* __restrict__ x, const uint4* __restrict__ gamma, const uint4* __restrict__ beta,
               float eps, int M, const int32_t* __restrict__ m_dev, int vec_per_row, uint4* __restrict__ out,
               const RowMapArgs maps, const LnModArgs mod)
{
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * kLnWarps + (threadIdx.x >> 5);
    if (m_dev) M = min(M, *m_dev);      // the host knows only an upper bound
    if (r >= M) return;
    long src = r;
    int img = 0;
    if (MOD && !MAPS) img = mod.img_row[r];
    if (MAPS) {
        // image of compacted row r: largest b with cu_keep[b] <= r
        int lo = 0, hi = maps.B;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (maps.cu_keep[mid] <= r) lo = mid; else hi = mid;
        }
        const int b = lo, c0 = maps.cu_keep[b];
        src = (long)b * maps.N + maps.keep_idx[r];
        img = b;
        if (lane == 0) {
            maps.src_row[r] = (int32_t)src;
            maps.img_row[r] = b;
            const int k_b = maps.cu_keep[b + 1] - c0, len = maps.kv_len[b];
            if (len + k_b > maps.Lmax) {
                maps.kv_row[r] = -1;
                atomicOr(maps.status, NOVA_DEV_SHAPE);
            } else {
                maps.kv_row[r] = b * maps.Lmax + len + (r - c0);
            }
        }
    }
    const uint4* xr = x + src * vec_per_row;
    // The row is read once (streaming loads, all issued before the first use) and stays in
    // registers for the three sweeps: sum, squared deviations, normalise.
    uint4 raw[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const int c = i * 32 + lane;
        raw[i] = (c < vec_per_row) ? ld_nc_stream(xr + c) : make_uint4(0, 0, 0, 0);
    }
    float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            sum0 += __uint_as_float(w[q] << 16);
            sum1 += __uint_as_float(w[q] & 0xffff0000u);
        }
    }
    const float n = (float)(vec_per_row * 8);
    const float mean = warp_sum(sum0 + sum1) / n;
    float sq0 = 0.f, sq1 = 0.f;
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        if (i * 32 + lane < vec_per_row) {
            const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float d0 = __uint_as_float(w[q] << 16) - mean, d1 = __uint_as_float(w[q] & 0xffff0000u) - mean;
                sq0 = fmaf(d0, d0, sq0);
                sq1 = fmaf(d1, d1, sq1);
            }
        }
    }
    const float rstd = rsqrtf(warp_sum(sq0 + sq1) / n + eps);
    const float shift = -mean * rstd;
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const int c = i * 32 + lane;
        if (c < vec_per_row) {
            const uint4 g = gamma[c], bt = beta[c];
            const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
            const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, bw[4] = {bt.x, bt.y, bt.z, bt.w};
            uint32_t o[4];
            uint32_t sc[4] = {0, 0, 0, 0}, sh[4] = {0, 0, 0, 0};        // bf16 zeros: no modulation
            if (MOD && mod.scale) { const uint4 t = mod.scale[(long)img * vec_per_row + c]; sc[0] = t.x; sc[1] = t.y; sc[2] = t.z; sc[3] = t.w; }
            if (MOD && mod.shift) { const uint4 t = mod.shift[(long)img * vec_per_row + c]; sh[0] = t.x; sh[1] = t.y; sh[2] = t.z; sh[3] = t.w; }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                // (x - mean) * rstd = x * rstd + shift
                const float n0 = fmaf(__uint_as_float(w[q] << 16), rstd, shift);
                const float n1 = fmaf(__uint_as_float(w[q] & 0xffff0000u), rstd, shift);
                float y0 = fmaf(n0, __uint_as_float(gw[q] << 16), __uint_as_float(bw[q] << 16));
                float y1 = fmaf(n1, __uint_as_float(gw[q] & 0xffff0000u), __uint_as_float(bw[q] & 0xffff0000u));
                if (MOD) {
                    y0 = fmaf(y0, 1.f + __uint_as_float(sc[q] << 16), __uint_as_float(sh[q] << 16));
                    y1 = fmaf(y1, 1.f + __uint_as_float(sc[q] & 0xffff0000u), __uint_as_float(sh[q] & 0xffff0000u));
                }
                __nv_bfloat162 t = __floats2bfloat162_rn(y0, y1);
                o[q] = *reinterpret_cast<uint32_t*>(&t);
            }
            out[(long)r * vec_per_row + c] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

// ---- query/key normalisation and rotary embedding -----------------------------------------------
// After the QKV projection, per kept row r and head: q (in the q buffer) and the row's new key (in
// its cache row) are, in place, scaled to unit L2 norm times a per-channel gain, then rotated pair by
// pair by the angle of the token's position in the scale. One warp per (row, head); a lane holds DH / 32
// consecutive channels, i.e. whole pairs.
template <int DH>
__global__ void __launch_bounds__(256)
qk_transform_kernel(__nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ k_cache, const int32_t* __restrict__ kv_row,
                    const int32_t* __restrict__ keep_idx, int M, const int32_t* __restrict__ m_dev, int C, int n_heads,
                    const __nv_bfloat16* __restrict__ gain_q, const __nv_bfloat16* __restrict__ gain_k, float eps,
                    const float* __restrict__ rope_cos, const float* __restrict__ rope_sin)
{
    constexpr int PER = DH / 32;          // 2 or 4 channels per lane
    const int lane = threadIdx.x & 31;
    const long wid = (long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (m_dev) M = min(M, *m_dev);
    if (wid >= (long)M * n_heads) return;
    const int r = (int)(wid / n_heads), hd = (int)(wid - (long)r * n_heads);
    const int pos = keep_idx[r];
    const int ch = hd * DH + lane * PER;
    float cs[PER / 2], sn[PER / 2];
    if (rope_cos) {
#pragma unroll
        for (int i = 0; i < PER / 2; ++i) {
            cs[i] = rope_cos[(long)pos * (DH / 2) + lane * (PER / 2) + i];
            sn[i] = rope_sin[(long)pos * (DH / 2) + lane * (PER / 2) + i];
        }
    }
    auto transform = [&](__nv_bfloat16* row, const __nv_bfloat16* gain) {
        float v[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) v[i] = __bfloat162float(row[ch + i]);
        if (gain) {
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < PER; ++i) ss = fmaf(v[i], v[i], ss);
            ss = warp_sum(ss);
            const float inv = 1.f / fmaxf(sqrtf(ss), eps);
#pragma unroll
            for (int i = 0; i < PER; ++i) v[i] = v[i] * inv * __bfloat162float(gain[ch + i]);
        }
        if (rope_cos) {
#pragma unroll
            for (int i = 0; i < PER / 2; ++i) {
                const float a = v[2 * i], b = v[2 * i + 1];
                v[2 * i] = a * cs[i] - b * sn[i];
                v[2 * i + 1] = a * sn[i] + b * cs[i];
            }
        }
#pragma unroll
        for (int i = 0; i < PER; ++i) row[ch + i] = __float2bfloat16_rn(v[i]);
    };
    transform(q + (long)r * C, gain_q);
    const int kr = kv_row[r];
    if (kr >= 0) transform(k_cache + (long)kr * C, gain_k);      // a row of an overflowing image has no cache row
}

struct Workspace {
    int32_t* src_row;
    int32_t* kv_row;
    int32_t* img_row;
    __nv_bfloat16 *h, *q, *o, *x1, *f;
    size_t bytes;
};

inline size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

Workspace carve(void* base, int M, int C, int F)
{
    Workspace w;
    size_t off = 0;
    auto take = [&](size_t bytes) { void* p = base ? (char*)base + off : nullptr; off += align_up(bytes); return p; };
    const size_t Mp = (size_t)((M + 127) / 128) * 128;   // whole 128-row tiles
    w.src_row = (int32_t*)take(Mp * 4);
    w.kv_row = (int32_t*)take(Mp * 4);
    w.h = (__nv_bfloat16*)take(Mp * C * 2);
    w.q = (__nv_bfloat16*)take(Mp * C * 2);
    w.o = (__nv_bfloat16*)take(Mp * C * 2);
    w.x1 = (__nv_bfloat16*)take(Mp * C * 2);
    w.f = (__nv_bfloat16*)take(Mp * (size_t)F * 2);
    w.img_row = (int32_t*)take(Mp * 4);
    w.bytes = off;
    return w;
}

bool shape_ok(const nova_block_shape* s)
{
    if (!s || s->B < 1 || s->N < 1 || s->C < 64 || s->n_heads < 1 || s->F < 64 || s->Lmax < 1 || s->M < 0) return false;
    if (s->C % 64 || s->F % 64 || s->C % s->n_heads) return false;
    const int dh = s->C / s->n_heads;
    if (dh != 64 && dh != 128) return false;
    if (s->C > 8192) return false;
    if ((long)s->M > (long)s->B * s->N) return false;
    return true;
}

}  // namespace

static nova_status launch_ln(nova_ctx* ctx, const __nv_bfloat16* x, const RowMapArgs* maps, const LnModArgs& mod,
                             const __nv_bfloat16* g, const __nv_bfloat16* b, float eps, int M, const int32_t* m_dev,
                             int C, __nv_bfloat16* out, cudaStream_t st)
{
    if (M <= 0) return NOVA_OK;
    const int vec = C / 8;
    const int per_lane = (vec + 31) / 32;
    const dim3 grid((M + kLnWarps - 1) / kLnWarps), block(kLnWarps * 32);
    RowMapArgs none;
    memset(&none, 0, sizeof(none));
    nova_launch_scope scope(ctx, NOVA_K_LAYERNORM, st);
#define NOVA_LN_LAUNCH(V, MAPS, MOD, MAPARG)                                                                     \
    layernorm_rows<V, MAPS, MOD><<<grid, block, 0, st>>>((const uint4*)x, (const uint4*)g, (const uint4*)b, eps, M, m_dev, vec, (uint4*)out, MAPARG, mod)
#define NOVA_LN_CASE(V)                                                                                          \
    do {                                                                                                         \
        if (maps && modulated) NOVA_LN_LAUNCH(V, true, true, *maps);                                             \
        else if (maps) NOVA_LN_LAUNCH(V, true, false, *maps);                                                    \
        else if (modulated) NOVA_LN_LAUNCH(V, false, true, none);                                                \
        else NOVA_LN_LAUNCH(V, false, false, none);                                                              \
    } while (0)
    const bool modulated = mod.scale || mod.shift;
    if (per_lane <= 2) NOVA_LN_CASE(2);
    else if (per_lane <= 4) NOVA_LN_CASE(4);
    else if (per_lane <= 8) NOVA_LN_CASE(8);
    else if (per_lane <= 16) NOVA_LN_CASE(16);
    else if (per_lane <= 32) NOVA_LN_CASE(32);
    else return nova_fail(ctx, NOVA_ERR_SHAPE, "layernorm: C > 8192");
#undef NOVA_LN_LAUNCH
#undef NOVA_LN_CASE
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

extern "C" size_t nova_block_workspace_bytes(const nova_block_shape* s)
{
    if (!shape_ok(s)) return 0;
    return carve(nullptr, s->M, s->C, s->F).bytes;
}

// Where the block's output goes when the last GEMM scatters it straight into the token map (Eq. 15-16
// on the kept rows) instead of writing the compacted y_kept.
struct ScatterOut {
    void* x_out;        // [B, N, C]: kept rows receive the layer output
    void* cache_out;    // [B, N, C] or NULL: kept rows receive output - input
};

// m_on_device: s->M is only an upper bound of the kept rows (it sizes grids, tensor maps and the
// workspace); every kernel takes the true count from cu_keep[B] on the device.
static nova_status block_forward(nova_ctx* ctx, const nova_block_weights* w, const nova_block_modulation* mod,
                                 const nova_block_shape* s, const void* x_in,
                                 const int32_t* keep_idx, const int32_t* cu_keep,
                                 void* k_cache, void* v_cache, int32_t* kv_len,
                                 int append_kv, void* y_kept, void* stream, bool m_on_device,
                                 const ScatterOut* scatter = nullptr, const nova_block_extras* ext = nullptr)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (!w || !s) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_block_forward: null weights or shape");
    if (!shape_ok(s)) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_pruned_block_forward: unsupported shape");
    if (s->M == 0) return NOVA_OK;
    if (!x_in || !keep_idx || !cu_keep || !k_cache || !v_cache || !kv_len || (!y_kept && !scatter))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_block_forward: null tensor");
    const void* wp[] = {w->ln1_g, w->ln1_b, w->w_qkv, w->b_qkv, w->w_o, w->b_o,
                        w->ln2_g, w->ln2_b, w->w_fc1, w->b_fc1, w->w_fc2, w->b_fc2};
    for (const void* ptr : wp) {
        if (!ptr) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_block_forward: null weight");
        if (!nova_aligned16(ptr)) return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_pruned_block_forward: weight not 16-byte aligned");
    }
    if (!nova_aligned16(x_in) || !nova_aligned16(k_cache) || !nova_aligned16(v_cache) || !nova_aligned16(y_kept))
        return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_pruned_block_forward: tensor not 16-byte aligned");
    Workspace ws = carve(ctx->workspace, s->M, s->C, s->F);
    if (!ctx->workspace || ctx->workspace_bytes < ws.bytes)
        return nova_fail(ctx, NOVA_ERR_WORKSPACE, "nova_pruned_block_forward: workspace missing or too small");
    const bool rope = ext && (ext->rope_cos || ext->rope_sin);
    const bool qk_norm = ext && (ext->qk_gain_q || ext->qk_gain_k);
    const bool cross = ext && ext->w_q2;
    if (rope && (!ext->rope_cos || !ext->rope_sin)) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_block_forward_ext: rope_cos and rope_sin go together");
    if (qk_norm && (!ext->qk_gain_q || !ext->qk_gain_k)) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_block_forward_ext: qk_gain_q and qk_gain_k go together");
    if (cross) {
        const void* cp[] = {ext->lnc_g, ext->lnc_b, ext->w_q2, ext->b_q2, ext->w_o2, ext->b_o2, ext->cond_k, ext->cond_v, ext->cond_len};
        for (const void* ptr : cp)
            if (!ptr) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_block_forward_ext: incomplete cross-attention weights");
        if (ext->Lc_max < 1) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_block_forward_ext: Lc_max < 1");
    }
    if (ext) {
        const void* ep[] = {ext->rope_cos, ext->rope_sin, ext->qk_gain_q, ext->qk_gain_k, ext->lnc_g, ext->lnc_b, ext->w_q2,
                            ext->b_q2, ext->w_o2, ext->b_o2, ext->cond_k, ext->cond_v};
        for (const void* ptr : ep)
            if (!nova_aligned16(ptr)) return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_pruned_block_forward_ext: tensor not 16-byte aligned");
    }
    NOVA_DEVICE_GUARD(ctx, "nova_pruned_block_forward");

    cudaStream_t st = (cudaStream_t)stream;
    {
        const nova_status chk = nova_debug_check_lists(ctx, "nova_pruned_block_forward", keep_idx, nullptr, cu_keep,
                                                       s->B, s->N, s->M, !m_on_device, st);
        if (chk != NOVA_OK) return chk;
    }
    const int M = s->M, C = s->C, F = s->F;
    typedef const __nv_bfloat16* cbf;
    typedef __nv_bfloat16* bf;

    const int32_t* m_dev = m_on_device ? cu_keep + s->B : nullptr;
    nova_block_modulation md;
    memset(&md, 0, sizeof(md));
    if (mod) md = *mod;
    const void* mp[] = {md.shift1, md.scale1, md.gate1, md.shift2, md.scale2, md.gate2};
    for (const void* ptr : mp)
        if (!nova_aligned16(ptr)) return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_pruned_block_forward: modulation not 16-byte aligned");
    LnModArgs ln1_mod = {(const uint4*)md.scale1, (const uint4*)md.shift1, ws.img_row};
    LnModArgs ln2_mod = {(const uint4*)md.scale2, (const uint4*)md.shift2, ws.img_row};
    nova_status rc;
    // h = LN1(gathered rows); the same kernel writes the row maps the GEMM epilogues use
    RowMapArgs maps;
    maps.keep_idx = keep_idx; maps.cu_keep = cu_keep; maps.kv_len = kv_len; maps.B = s->B; maps.N = s->N;
    maps.Lmax = s->Lmax; maps.src_row = ws.src_row; maps.kv_row = ws.kv_row; maps.img_row = ws.img_row; maps.status = ctx->dev_status;
    rc = launch_ln(ctx, (cbf)x_in, &maps, ln1_mod, (cbf)w->ln1_g, (cbf)w->ln1_b, w->eps, M, m_dev, C, ws.h, st);
    if (rc) return rc;
    // [q | k | v] = h W_qkv^T + b; k, v go straight to their cache rows
    nova_gemm_args g;
    memset(&g, 0, sizeof(g));
    g.A = ws.h; g.W = (cbf)w->w_qkv; g.bias = (cbf)w->b_qkv; g.M = M; g.m_dev = m_dev; g.N = 3 * C; g.K = C;
    g.epilogue = NOVA_EPI_QKV; g.cat = NOVA_K_GEMM_QKV; g.out = ws.q; g.C = C; g.k_cache = (bf)k_cache; g.v_cache = (bf)v_cache; g.kv_row = ws.kv_row;
    rc = nova_launch_gemm(ctx, g, st);
    if (rc) return rc;
    if (rope || qk_norm) {
        // q and the new keys, in place: unit norm times gain, then the rotation of the token's position
        const long warps = (long)M * s->n_heads;
        const unsigned blocks = (unsigned)((warps + 7) / 8);
        typedef const float* cfl;
        nova_launch_scope scope(ctx, NOVA_K_LAYERNORM, st);
        if (C / s->n_heads == 64)
            qk_transform_kernel<64><<<blocks, 256, 0, st>>>(ws.q, (bf)k_cache, ws.kv_row, keep_idx, M, m_dev, C, s->n_heads,
                                                          (cbf)ext->qk_gain_q, (cbf)ext->qk_gain_k, ext->qk_eps,
                                                          (cfl)ext->rope_cos, (cfl)ext->rope_sin);
        else
            qk_transform_kernel<128><<<blocks, 256, 0, st>>>(ws.q, (bf)k_cache, ws.kv_row, keep_idx, M, m_dev, C, s->n_heads,
                                                           (cbf)ext->qk_gain_q, (cbf)ext->qk_gain_k, ext->qk_eps,
                                                           (cfl)ext->rope_cos, (cfl)ext->rope_sin);
        NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    }
    // o = softmax(q K^T / sqrt(dh)) V
    nova_attn_args a;
    a.q = ws.q; a.k_cache = (cbf)k_cache; a.v_cache = (cbf)v_cache; a.cu_keep = cu_keep; a.kv_len = kv_len;
    a.o = ws.o; a.B = s->B; a.C = C; a.n_heads = s->n_heads; a.Lmax = s->Lmax; a.M = M;
    // neither the projection's output buffer nor the MLP's hidden buffer is in use yet, and they lie
    // next to each other: together they hold the partial results of a key-split last wave
    a.scratch = ws.x1;
    a.scratch_bytes = (size_t)((char*)ws.f - (char*)ws.x1) + (size_t)((M + 127) / 128) * 128 * (size_t)F * 2;
    a.cache_only = false;
    rc = nova_launch_attention(ctx, a, st);
    if (rc) return rc;
    // x1 = Xc + o W_o^T + b_o
    memset(&g, 0, sizeof(g));
    g.A = ws.o; g.W = (cbf)w->w_o; g.bias = (cbf)w->b_o; g.M = M; g.m_dev = m_dev; g.N = C; g.K = C;
    g.epilogue = NOVA_EPI_BIAS_RES; g.cat = NOVA_K_GEMM_PROJ; g.out = ws.x1; g.res = (cbf)x_in; g.res_row = ws.src_row;
    g.gate = (cbf)md.gate1; g.img_row = ws.img_row;
    rc = nova_launch_gemm(ctx, g, st);
    if (rc) return rc;
    if (cross) {
        // x1 <- x1 + softmax(q2 Kc^T / sqrt(dh)) Vc W_o2^T + b_o2 with q2 = LN(x1) W_q2^T + b_q2: the same
        // kernels once more, on buffers that are free at this point (h, q, o), the keys and values being
        // the image's condition tokens and nothing else
        LnModArgs none_mod = {nullptr, nullptr, ws.img_row};
        rc = launch_ln(ctx, ws.x1, nullptr, none_mod, (cbf)ext->lnc_g, (cbf)ext->lnc_b, w->eps, M, m_dev, C, ws.h, st);
        if (rc) return rc;
        memset(&g, 0, sizeof(g));
        g.A = ws.h; g.W = (cbf)ext->w_q2; g.bias = (cbf)ext->b_q2; g.M = M; g.m_dev = m_dev; g.N = C; g.K = C;
        g.epilogue = NOVA_EPI_QKV; g.cat = NOVA_K_GEMM_QKV; g.out = ws.q; g.C = C; g.kv_row = ws.kv_row;   // all columns are q
        rc = nova_launch_gemm(ctx, g, st);
        if (rc) return rc;
        nova_attn_args ca;
        ca.q = ws.q; ca.k_cache = (cbf)ext->cond_k; ca.v_cache = (cbf)ext->cond_v; ca.cu_keep = cu_keep; ca.kv_len = ext->cond_len;
        ca.o = ws.o; ca.B = s->B; ca.C = C; ca.n_heads = s->n_heads; ca.Lmax = ext->Lc_max; ca.M = M;
        ca.scratch = nullptr; ca.scratch_bytes = 0;      // x1 is live: no room for a key-split wave
        ca.cache_only = true;
        rc = nova_launch_attention(ctx, ca, st);
        if (rc) return rc;
        memset(&g, 0, sizeof(g));
        g.A = ws.o; g.W = (cbf)ext->w_o2; g.bias = (cbf)ext->b_o2; g.M = M; g.m_dev = m_dev; g.N = C; g.K = C;
        g.epilogue = NOVA_EPI_BIAS_RES; g.cat = NOVA_K_GEMM_PROJ; g.out = ws.x1; g.res = ws.x1; g.res_row = nullptr;   // in place
        rc = nova_launch_gemm(ctx, g, st);
        if (rc) return rc;
    }
    // h = LN2(x1)
    rc = launch_ln(ctx, ws.x1, nullptr, ln2_mod, (cbf)w->ln2_g, (cbf)w->ln2_b, w->eps, M, m_dev, C, ws.h, st);
    if (rc) return rc;
    // f = GELU(h W_fc1^T + b_fc1)
    memset(&g, 0, sizeof(g));
    g.A = ws.h; g.W = (cbf)w->w_fc1; g.bias = (cbf)w->b_fc1; g.M = M; g.m_dev = m_dev; g.N = F; g.K = C;
    g.epilogue = NOVA_EPI_BIAS_GELU; g.cat = NOVA_K_GEMM_FC1; g.out = ws.f;
    rc = nova_launch_gemm(ctx, g, st);
    if (rc) return rc;
    // y = x1 + f W_fc2^T + b_fc2
    memset(&g, 0, sizeof(g));
    g.A = ws.f; g.W = (cbf)w->w_fc2; g.bias = (cbf)w->b_fc2; g.M = M; g.m_dev = m_dev; g.N = C; g.K = F;
    g.epilogue = NOVA_EPI_BIAS_RES; g.cat = NOVA_K_GEMM_FC2; g.out = (bf)y_kept; g.res = ws.x1; g.res_row = nullptr;
    g.gate = (cbf)md.gate2; g.img_row = ws.img_row;
    if (scatter) {
        // kept row r is token src_row[r] of the map: x_out[token] = y, cache_out[token] = y - x_in[token]
        g.out = (bf)scatter->x_out; g.out_row = ws.src_row;
        g.diff_in = (cbf)x_in; g.diff_out = (bf)scatter->cache_out;
    }
    if (append_kv) {
        // the last kernel of the block also advances kv_len: every reader of the old lengths (row
        // maps, attention) ran in an earlier kernel of this call
        g.adv_cu_keep = cu_keep; g.adv_kv_len = kv_len; g.adv_B = s->B; g.adv_Lmax = s->Lmax;
    }
    rc = nova_launch_gemm(ctx, g, st);
    if (rc) return rc;
    return NOVA_OK;
}

extern "C" nova_status nova_pruned_block_forward(nova_ctx* ctx, const nova_block_weights* w,
                                                 const nova_block_shape* s, const void* x_in,
                                                 const int32_t* keep_idx, const int32_t* cu_keep,
                                                 void* k_cache, void* v_cache, int32_t* kv_len,
                                                 int append_kv, void* y_kept, void* stream)
{
    return block_forward(ctx, w, nullptr, s, x_in, keep_idx, cu_keep, k_cache, v_cache, kv_len, append_kv, y_kept, stream, false);
}

extern "C" nova_status nova_pruned_block_forward_device(nova_ctx* ctx, const nova_block_weights* w,
                                                        const nova_block_shape* s, const void* x_in,
                                                        const int32_t* keep_idx, const int32_t* cu_keep,
                                                        void* k_cache, void* v_cache, int32_t* kv_len,
                                                        int append_kv, void* y_kept, void* stream)
{
    return block_forward(ctx, w, nullptr, s, x_in, keep_idx, cu_keep, k_cache, v_cache, kv_len, append_kv, y_kept, stream, true);
}

extern "C" nova_status nova_pruned_block_forward_adaln(nova_ctx* ctx, const nova_block_weights* w,
                                                       const nova_block_modulation* mod,
                                                       const nova_block_shape* s, const void* x_in,
                                                       const int32_t* keep_idx, const int32_t* cu_keep,
                                                       void* k_cache, void* v_cache, int32_t* kv_len,
                                                       int append_kv, void* y_kept, int m_on_device, void* stream)
{
    return block_forward(ctx, w, mod, s, x_in, keep_idx, cu_keep, k_cache, v_cache, kv_len, append_kv, y_kept, stream,
                         m_on_device != 0);
}

extern "C" nova_status nova_pruned_block_forward_ext(nova_ctx* ctx, const nova_block_weights* w,
                                                     const nova_block_modulation* mod, const nova_block_extras* ext,
                                                     const nova_block_shape* s, const void* x_in,
                                                     const int32_t* keep_idx, const int32_t* cu_keep,
                                                     void* k_cache, void* v_cache, int32_t* kv_len,
                                                     int append_kv, void* y_kept, int m_on_device, void* stream)
{
    return block_forward(ctx, w, mod, s, x_in, keep_idx, cu_keep, k_cache, v_cache, kv_len, append_kv, y_kept, stream,
                         m_on_device != 0, nullptr, ext);
}

// Eq. 14 followed by Eq. 15-16 for one layer: the block on the kept rows with its last GEMM writing
// the kept rows of x_out / cache_out directly, then the pruned rows from the upsampled cache.
extern "C" nova_status nova_pruned_layer_forward(nova_ctx* ctx, const nova_block_weights* w,
                                                 const nova_block_modulation* mod, const nova_block_shape* s,
                                                 const void* x_in, const int32_t* keep_idx, const int32_t* prune_idx,
                                                 const int32_t* cu_keep, void* k_cache, void* v_cache, int32_t* kv_len,
                                                 int append_kv, const void* cache_prev, int hp, int wp, int h, int w_,
                                                 void* x_out, void* cache_out, int m_on_device, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (!s) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_layer_forward: null shape");
    if (!shape_ok(s)) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_pruned_layer_forward: unsupported shape");
    if ((long)h * w_ != (long)s->N) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_layer_forward: h * w must equal N");
    if (!x_in || !x_out || !cu_keep) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_layer_forward: null tensor");
    if (x_out == x_in) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_layer_forward: x_out aliases x_in");
    if (!nova_aligned16(x_out) || !nova_aligned16(cache_out))
        return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_pruned_layer_forward: tensors must be 16-byte aligned");
    const long total = (long)s->B * s->N;
    if (total > 0x7fffffffL) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_pruned_layer_forward: too many rows");
    const bool on_dev = m_on_device != 0;
    if ((s->M < total || on_dev) && (!prune_idx || !cache_prev || hp < 1 || wp < 1))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_layer_forward: pruned rows need prune_idx and cache_prev");
    NOVA_DEVICE_GUARD(ctx, "nova_pruned_layer_forward");
    {   // debug mode: both lists are checked before the block's first kernel, so that a bad pruned list leaves no half-done layer
        const nova_status chk = nova_debug_check_lists(ctx, "nova_pruned_layer_forward", keep_idx, prune_idx, cu_keep,
                                                       s->B, s->N, s->M, !on_dev, (cudaStream_t)stream);
        if (chk != NOVA_OK) return chk;
    }
    ScatterOut sc = {x_out, cache_out};
    nova_status rc = block_forward(ctx, w, mod, s, x_in, keep_idx, cu_keep, k_cache, v_cache, kv_len, append_kv, nullptr,
                                   stream, on_dev, &sc);
    if (rc != NOVA_OK) return rc;
    return nova_restore_pruned_rows(ctx, x_in, prune_idx, cu_keep, cache_prev, hp, wp, h, w_, s->C, s->B, s->M, on_dev,
                                    x_out, cache_out, stream);
}

// ---- block forward for callers that cannot allocate device memory --------------------------
// The scratch that nova_pruned_block_forward normally takes from the caller's workspace lives
// here, in a fixed array that is part of the library image: every GPU that loads the library
// holds these bytes until the process exits.
#define NOVA_STATIC_SCRATCH_BYTES (6u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[NOVA_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch per CUDA device ordinal. In host code the array's name is
// only a handle for the runtime, not an address a kernel can use; the real address is looked up
// once per device with that device current.
static void* g_static_scratch_addr[64];

extern "C" size_t nova_static_scratch_bytes(void) { return NOVA_STATIC_SCRATCH_BYTES; }

extern "C" nova_status nova_pruned_block_forward_static(nova_ctx* ctx, const nova_block_weights* w,
                                                        const nova_block_shape* s, const void* x_in,
                                                        const int32_t* keep_idx, const int32_t* cu_keep,
                                                        void* k_cache, void* v_cache, int32_t* kv_len,
                                                        int append_kv, void* y_kept, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (!s) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_pruned_block_forward_static: null shape");
    if (ctx->profiling)
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG,
                         "nova_pruned_block_forward_static: not available inside a profiling window (event creation may allocate)");
    if (!shape_ok(s)) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_pruned_block_forward_static: unsupported shape");
    if (s->M == 0) return NOVA_OK;      // nothing kept: a no-op, as for the ordinary entry point
    const size_t need = nova_block_workspace_bytes(s);
    if (need > NOVA_STATIC_SCRATCH_BYTES) {
        snprintf(ctx->err, sizeof(ctx->err),
                 "nova_pruned_block_forward_static: shape needs %zu bytes of scratch, the built-in array holds %u",
                 need, (unsigned)NOVA_STATIC_SCRATCH_BYTES);
        return NOVA_ERR_WORKSPACE;
    }
    int cur = -1;
    NOVA_CUDA_CHECK(ctx, cudaGetDevice(&cur));
    if (cur != ctx->device || cur < 0 || cur >= 64)
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG,
                         "nova_pruned_block_forward_static: the context's device must be the current device");
    if (!g_static_scratch_addr[cur]) {
        void* addr = nullptr;
        NOVA_CUDA_CHECK(ctx, cudaGetSymbolAddress(&addr, g_static_scratch));
        g_static_scratch_addr[cur] = addr;
    }
    // Run the ordinary path with the built-in array standing in for the caller's workspace.
    void* saved_ws = ctx->workspace;
    const size_t saved_bytes = ctx->workspace_bytes;
    ctx->workspace = g_static_scratch_addr[cur];
    ctx->workspace_bytes = NOVA_STATIC_SCRATCH_BYTES;
    const nova_status rc = nova_pruned_block_forward(ctx, w, s, x_in, keep_idx, cu_keep, k_cache, v_cache, kv_len,
                                                     append_kv, y_kept, stream);
    ctx->workspace = saved_ws;
    ctx->workspace_bytes = saved_bytes;
    return rc;
}

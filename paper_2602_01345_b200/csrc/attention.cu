// Attention of the kept queries over [prior-scale K/V cache ++ kept tokens' own K/V]
// (no mask), on the sm_100a tensor cores.
//
// One CTA = 128 query rows of one image and one head. Streaming (flash-style) softmax:
//   warp 0      TMA producer: Q once, then a 2-stage ring of {K tile, V tile} (128 keys each)
//   warp 1      tcgen05.mma issuer:  S = Q K^T  (fp32 in TMEM, double buffered)
//                                    O_tile = P V (fp32 in TMEM)
//   warps 2-5   one query row per thread: read S from TMEM, running max / sum, write
//               P = exp2(...) as bf16 into shared memory in the swizzled K-major layout the
//               tensor core reads, then fold O_tile into the fp32 output registers.
// K tiles are K-major operands; V tiles are used as the MN-major B operand of P V, so V is
// consumed exactly as it lies in the cache ([keys, dh] row-major).
// Every mbarrier wait is bounded.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BQ = 128;        // query rows per CTA
constexpr int BKV = 128;       // keys per tile
constexpr int kThreads = 192;
constexpr int kSlabBytes = 128 * 128;   // [128 rows][64 bf16]
constexpr int kKvStages = 2;

template <int DH>
struct AttnSmem {
    static constexpr int kSlabs = DH / 64;
    static constexpr int kQBytes = kSlabs * kSlabBytes;
    static constexpr int kKBytes = kSlabs * kSlabBytes;
    static constexpr int kVBytes = kSlabs * kSlabBytes;
    static constexpr int kPBytes = 2 * kSlabBytes;
    static constexpr int kQOff = 0;
    static constexpr int kKOff = kQBytes;
    static constexpr int kVOff = kKOff + kKvStages * kKBytes;
    static constexpr int kPOff = kVOff + kKvStages * kVBytes;
    static constexpr int kBarOff = kPOff + kPBytes;
    static constexpr int kTotal = kBarOff + 256 + 1024;
};

struct AttnParams {
    const int32_t* cu_keep;
    const int32_t* kv_len;
    __nv_bfloat16* o;
    int B, C, Lmax;
    float scale_log2e;     // (1 / sqrt(dh)) * log2(e)
    unsigned int* status;
};

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

template <int DH>
__global__ void __launch_bounds__(kThreads)
attention_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                 const __grid_constant__ CUtensorMap tmap_v, const AttnParams p)
{
    using L = AttnSmem<DH>;
    constexpr int kSlabs = L::kSlabs;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColS0 = 0, kColS1 = 128, kColO = 256;

    // ---- which (image, query tile) is this CTA? ------------------------------------
    int slot = blockIdx.x, b = 0, k_b = 0, q_begin = 0;
    bool found = false;
    for (b = 0; b < p.B; ++b) {
        const int c0 = p.cu_keep[b];
        k_b = p.cu_keep[b + 1] - c0;
        const int tiles = (k_b + BQ - 1) / BQ;
        if (slot < tiles) { q_begin = c0 + slot * BQ; found = true; break; }
        slot -= tiles;
    }
    if (!found) return;
    const int rows_valid = min(BQ, k_b - slot * BQ);
    const int head = blockIdx.y;
    const int n_keys = min(p.kv_len[b] + k_b, p.Lmax);
    const int n_tiles = (n_keys + BKV - 1) / BKV;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = (uint64_t*)(smem + L::kBarOff);
    uint64_t* q_full = bars;            // 1
    uint64_t* k_full = bars + 1;        // 2
    uint64_t* v_full = bars + 3;        // 2
    uint64_t* kv_empty = bars + 5;      // 2
    uint64_t* s_full = bars + 7;        // 2
    uint64_t* p_full = bars + 9;        // 1 (128 arrivals)
    uint64_t* o_full = bars + 10;       // 1
    uint32_t* tmem_slot = (uint32_t*)(bars + 11);
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        mbar_init(q_full, 1);
        for (int s = 0; s < kKvStages; ++s) {
            mbar_init(&k_full[s], 1);
            mbar_init(&v_full[s], 1);
            mbar_init(&kv_empty[s], 1);
            mbar_init(&s_full[s], 1);
        }
        mbar_init(p_full, 128);
        mbar_init(o_full, 1);
        fence_barrier_init();
        prefetch_tmap(&tmap_q);
        prefetch_tmap(&tmap_k);
        prefetch_tmap(&tmap_v);
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    uint8_t* q_smem = smem + L::kQOff;
    uint8_t* p_smem = smem + L::kPOff;

    if (warp == 0) {
        if (lane == 0) {
            mbar_arrive_expect_tx(q_full, L::kQBytes);
            for (int sl = 0; sl < kSlabs; ++sl)
                tma_load_2d(q_smem + sl * kSlabBytes, &tmap_q, q_full, head * DH + sl * 64, q_begin);
            int issued = 0;
            for (int j = 0; j < n_tiles; ++j) {
                const int s = j % kKvStages;
                if (j >= kKvStages && !mbar_wait(&kv_empty[s], ((j / kKvStages) - 1) & 1, abort_flag, p.status)) break;
                uint8_t* k_dst = smem + L::kKOff + s * L::kKBytes;
                uint8_t* v_dst = smem + L::kVOff + s * L::kVBytes;
                mbar_arrive_expect_tx(&k_full[s], L::kKBytes);
                for (int sl = 0; sl < kSlabs; ++sl)
                    tma_load_3d(k_dst + sl * kSlabBytes, &tmap_k, &k_full[s], head * DH + sl * 64, j * BKV, b);
                mbar_arrive_expect_tx(&v_full[s], L::kVBytes);
                for (int sl = 0; sl < kSlabs; ++sl)
                    tma_load_3d(v_dst + sl * kSlabBytes, &tmap_v, &v_full[s], head * DH + sl * 64, j * BKV, b);
                issued = j + 1;
            }
            if (*abort_flag) {
                mbar_drain(q_full, 0);
                for (int j = max(0, issued - kKvStages); j < issued; ++j) {
                    mbar_drain(&k_full[j % kKvStages], (j / kKvStages) & 1);
                    mbar_drain(&v_full[j % kKvStages], (j / kKvStages) & 1);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_s = idesc_bf16_f32(BQ, BKV, 0);
            constexpr uint32_t idesc_o = idesc_bf16_f32(BQ, DH, 1);
            const uint32_t q_addr = smem_u32(q_smem), p_addr = smem_u32(p_smem);
            bool ok = mbar_wait(q_full, 0, abort_flag, p.status);
            auto issue_s = [&](int j) -> bool {
                const int s = j % kKvStages;
                if (!mbar_wait(&k_full[s], (j / kKvStages) & 1, abort_flag, p.status)) return false;
                tc_fence_after();
                const uint32_t k_addr = smem_u32(smem + L::kKOff + s * L::kKBytes);
                const uint32_t d = tmem_base + ((j & 1) ? kColS1 : kColS0);
#pragma unroll
                for (int kk = 0; kk < DH / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kSlabBytes + (kk & 3) * 32;
                    mma_bf16_ss(d, smem_desc_sw128(q_addr + off, 16, 1024), smem_desc_sw128(k_addr + off, 16, 1024),
                                idesc_s, kk ? 1u : 0u);
                }
                mma_commit(&s_full[j & 1]);
                return true;
            };
            if (ok) ok = issue_s(0);
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int s = j % kKvStages;
                if (j + 1 < n_tiles) { ok = issue_s(j + 1); if (!ok) break; }
                ok = mbar_wait(p_full, j & 1, abort_flag, p.status) &&
                     mbar_wait(&v_full[s], (j / kKvStages) & 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t v_addr = smem_u32(smem + L::kVOff + s * L::kVBytes);
#pragma unroll
                for (int kk = 0; kk < BKV / 16; ++kk) {
                    // A = P: K-major, 16 keys = 32 bytes inside a 64-key slab
                    const uint64_t adesc = smem_desc_sw128(p_addr + (kk >> 2) * kSlabBytes + (kk & 3) * 32, 16, 1024);
                    // B = V: MN-major (dh contiguous); 16 keys = 16 rows of 128 bytes; the next
                    // 64 dh columns live one slab further (leading byte offset)
                    const uint64_t bdesc = smem_desc_sw128(v_addr + kk * 2048, kSlabBytes, 1024);
                    mma_bf16_ss(tmem_base + kColO, adesc, bdesc, idesc_o, kk ? 1u : 0u);
                }
                mma_commit(o_full);
                mma_commit(&kv_empty[s]);
            }
        }
    } else {
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        float o_acc[DH];
#pragma unroll
        for (int i = 0; i < DH; ++i) o_acc[i] = 0.f;
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
            ok = mbar_wait_warp(&s_full[j & 1], (j >> 1) & 1, abort_flag, p.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t s_addr = tmem_base + lane_off + ((j & 1) ? kColS1 : kColS0);
            const int cols_valid = min(BKV, n_keys - j * BKV);
            // pass 1: row maximum over the valid keys
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < BKV / 32; ++c) {
                uint32_t sv[32];
                tmem_ld32(s_addr + c * 32, sv);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (c * 32 + i < cols_valid) mx = fmaxf(mx, __uint_as_float(sv[i]));
            }
            const float m_new = fmaxf(m_run, mx);
            const float alpha = ex2((m_run - m_new) * p.scale_log2e);
            const float m_scaled = m_new * p.scale_log2e;
            // pass 2: probabilities -> bf16 -> shared memory (row `row`, 128-byte swizzle)
            float lsum = 0.f;
            uint8_t* p_row = p_smem + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll 1
            for (int c = 0; c < BKV / 32; ++c) {
                uint32_t sv[32];
                tmem_ld32(s_addr + c * 32, sv);
                tmem_ld_wait();
                float pv[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float e = ex2(fmaf(__uint_as_float(sv[i]), p.scale_log2e, -m_scaled));
                    pv[i] = (c * 32 + i < cols_valid) ? e : 0.f;
                    lsum += pv[i];
                }
                uint8_t* slab = p_row + (c >> 1) * kSlabBytes;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int chunk16 = (c & 1) * 4 + g;
                    uint4 val = make_uint4(pack_bf16(pv[g * 8], pv[g * 8 + 1]), pack_bf16(pv[g * 8 + 2], pv[g * 8 + 3]),
                                           pack_bf16(pv[g * 8 + 4], pv[g * 8 + 5]), pack_bf16(pv[g * 8 + 6], pv[g * 8 + 7]));
                    *(uint4*)(slab + ((chunk16 ^ (row & 7)) << 4)) = val;
                }
            }
            l_run = l_run * alpha + lsum;
            m_run = m_new;
            if (cols_valid < BKV) {
                // ragged last tile: rows of V past the last key may hold anything (even NaN);
                // zero them so that 0 * garbage cannot poison the accumulator
                const int s = j % kKvStages;
                ok = mbar_wait_warp(&v_full[s], (j / kKvStages) & 1, abort_flag, p.status);
                if (!ok) break;
                if (row >= cols_valid) {
                    uint8_t* v_row = smem + L::kVOff + s * L::kVBytes + row * 128;
#pragma unroll
                    for (int sl = 0; sl < kSlabs; ++sl)
#pragma unroll
                        for (int g = 0; g < 8; ++g) *(uint4*)(v_row + sl * kSlabBytes + g * 16) = make_uint4(0, 0, 0, 0);
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(p_full);
            // fold this tile's P V into the running output
            ok = mbar_wait_warp(o_full, j & 1, abort_flag, p.status);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < DH / 32; ++c) {
                uint32_t ov[32];
                tmem_ld32(tmem_base + lane_off + kColO + c * 32, ov);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) o_acc[c * 32 + i] = fmaf(o_acc[c * 32 + i], alpha, __uint_as_float(ov[i]));
            }
            tc_fence_before();
        }
        if (ok && row < rows_valid) {
            const float inv = 1.f / l_run;
            uint4* dst = (uint4*)(p.o + (long)(q_begin + row) * p.C + head * DH);
#pragma unroll
            for (int g = 0; g < DH / 8; ++g)
                dst[g] = make_uint4(pack_bf16(o_acc[g * 8] * inv, o_acc[g * 8 + 1] * inv),
                                    pack_bf16(o_acc[g * 8 + 2] * inv, o_acc[g * 8 + 3] * inv),
                                    pack_bf16(o_acc[g * 8 + 4] * inv, o_acc[g * 8 + 5] * inv),
                                    pack_bf16(o_acc[g * 8 + 6] * inv, o_acc[g * 8 + 7] * inv));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

template <int DH>
nova_status launch(nova_ctx* ctx, const nova_attn_args& a, cudaStream_t st)
{
    using L = AttnSmem<DH>;
    CUtensorMap tq, tk, tv;
    const uint64_t dq[2] = {(uint64_t)a.C, (uint64_t)a.M}, sq[1] = {(uint64_t)a.C * 2};
    const uint64_t dk[3] = {(uint64_t)a.C, (uint64_t)a.Lmax, (uint64_t)a.B};
    const uint64_t sk[2] = {(uint64_t)a.C * 2, (uint64_t)a.Lmax * a.C * 2};
    if (!make_tmap_bf16(ctx, &tq, a.q, 2, dq, sq, BQ) || !make_tmap_bf16(ctx, &tk, a.k_cache, 3, dk, sk, BKV) ||
        !make_tmap_bf16(ctx, &tv, a.v_cache, 3, dk, sk, BKV))
        return nova_fail(ctx, NOVA_ERR_CUDA, "attention: cuTensorMapEncodeTiled failed");
    auto kern = attention_kernel<DH>;
    if (!ctx->attr_attn) {   // both head sizes opt in once per context
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<64>::kTotal));
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<128>::kTotal));
        ctx->attr_attn = true;
    }
    AttnParams p;
    p.cu_keep = a.cu_keep; p.kv_len = a.kv_len; p.o = a.o; p.B = a.B; p.C = a.C; p.Lmax = a.Lmax;
    p.scale_log2e = (float)((1.0 / sqrt((double)DH)) * 1.4426950408889634);
    p.status = ctx->dev_status;
    dim3 grid((a.M + BQ - 1) / BQ + a.B, a.n_heads);
    {
        nova_launch_scope scope(ctx, NOVA_K_ATTENTION, st);
        kern<<<grid, kThreads, L::kTotal, st>>>(tq, tk, tv, p);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

}  // namespace

nova_status nova_launch_attention(nova_ctx* ctx, const nova_attn_args& a, cudaStream_t st)
{
    if (a.M <= 0) return NOVA_OK;
    const int dh = a.C / a.n_heads;
    if (dh == 64) return launch<64>(ctx, a, st);
    if (dh == 128) return launch<128>(ctx, a, st);
    return nova_fail(ctx, NOVA_ERR_SHAPE, "attention: head dimension must be 64 or 128");
}

// out[M, N] = epilogue(A[M, K] * W[N, K]^T + bias) on the sm_100a tensor cores.
//
// Both operands are K-major bf16, so one TMA box of 64 K-elements (128 bytes, 128-byte
// swizzle) per row feeds tcgen05.mma directly. One CTA computes one 128 x BN output tile:
//   warp 0      TMA producer: fills a ring of kStages {A tile, W tile} buffers
//   warp 1      allocates TMEM, issues tcgen05.mma (one elected thread), commits to mbarriers
//   warps 2-5   epilogue: tcgen05.ld the fp32 accumulator (one row per thread), add bias,
//               apply GELU / residual / QKV routing, store bf16
// Large problems run on a second kernel, gemm_bf16_tn_pair: a persistent grid of CTA pairs
// (clusters of two, tcgen05 cta_group::2), each pair computing 256 x BN tiles. Per tensor-core
// instruction each CTA supplies only its 128 rows of A and BN/2 rows of W, which halves the
// shared-memory and L2 traffic per flop of the single-CTA tile; the fp32 accumulator is double
// buffered in tensor memory so that the epilogue of tile i overlaps the main loop of tile i+1, and
// eight epilogue warps (two per tensor-memory lane quarter, alternate column chunks) keep the
// epilogue shorter than the main loop even with GELU.
// Every mbarrier wait is bounded; on expiry the CTA records a timeout and tears down.
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kThreads = 192;

template <int BN, int STAGES>
struct GemmSmem {
    static constexpr int kABytes = BM * BK * 2;
    static constexpr int kBBytes = BN * BK * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTotal = STAGES * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

__device__ __forceinline__ float gelu_tanh(float x)
{
    // 0.5 x (1 + tanh(c (x + 0.044715 x^3))) with the hardware tanh (relative error 2^-11, an order
    // of magnitude below the bf16 rounding of the result): six instructions per element. The FC1
    // epilogue is bound by its instruction count, not by memory.
    const float c = 0.7978845608028654f;
    const float inner = x * fmaf(x * x, 0.044715f * c, c);
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(inner));
    const float hx = 0.5f * x;
    return fmaf(hx, t, hx);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

struct GemmParams {
    const __nv_bfloat16* bias;
    int M, N, K;
    int epilogue;
    __nv_bfloat16* out;
    const __nv_bfloat16* res;
    const int32_t* res_row;
    int C;
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    const int32_t* kv_row;
    unsigned int* status;
    const int32_t* adv_cu_keep;
    int32_t* adv_kv_len;
    int adv_B, adv_Lmax;
    float* ent;
    const int32_t* m_dev;
    const __nv_bfloat16* gate;
    const int32_t* img_row;
    const int32_t* out_row;
    const __nv_bfloat16* diff_in;
    __nv_bfloat16* diff_out;
};

// Rows of this launch: p.M, or the device-side count when the host only knows an upper bound.
__device__ __forceinline__ int true_rows(const GemmParams& p)
{
    return p.m_dev ? min(max(*p.m_dev, 0), p.M) : p.M;
}

// Advance of the K/V cache lengths, done by one warp-sized loop of the launch's first CTA.
__device__ __forceinline__ void advance_kv_len(const GemmParams& p)
{
    if (!p.adv_kv_len) return;
    for (int b = threadIdx.x; b < p.adv_B; b += blockDim.x) {
        const int k_b = p.adv_cu_keep[b + 1] - p.adv_cu_keep[b];
        if (p.adv_kv_len[b] + k_b <= p.adv_Lmax) p.adv_kv_len[b] += k_b;
    }
}


// Epilogue of 32 consecutive accumulator columns [col0, col0 + 32) of output row `row`:
// + bias, then GELU / residual / QKV routing, rounded to bf16 and stored with 128-bit stores.
__device__ __forceinline__ void epilogue_chunk(const GemmParams& p, int row, int col0, const uint32_t (&acc)[32],
                                               long res_base, long kv_base)
{
    float v[32];
    const uint4* bias4 = (const uint4*)(p.bias + col0);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 b = bias4[i];
        const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            v[i * 8 + j * 2] = __uint_as_float(acc[i * 8 + j * 2]) + __uint_as_float(bw[j] << 16);
            v[i * 8 + j * 2 + 1] = __uint_as_float(acc[i * 8 + j * 2 + 1]) + __uint_as_float(bw[j] & 0xffff0000u);
        }
    }
    __nv_bfloat16* dst;
    if (p.epilogue == NOVA_EPI_BIAS_GELU) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = gelu_tanh(v[i]);
        dst = p.out + (long)row * p.N + col0;
    } else if (p.epilogue == NOVA_EPI_BIAS_RES) {
        if (p.gate) {
            // per-image gate of the branch: out = residual + gate * (acc + bias)
            const uint4* g4 = (const uint4*)(p.gate + (long)p.img_row[row] * p.N + col0);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 g = g4[i];
                const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    v[i * 8 + j * 2] *= __uint_as_float(gw[j] << 16);
                    v[i * 8 + j * 2 + 1] *= __uint_as_float(gw[j] & 0xffff0000u);
                }
            }
        }
        const uint4* r4 = (const uint4*)(p.res + res_base + col0);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 r = r4[i];
            const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[i * 8 + j * 2] += __uint_as_float(rw[j] << 16);
                v[i * 8 + j * 2 + 1] += __uint_as_float(rw[j] & 0xffff0000u);
            }
        }
        const long orow = p.out_row ? (long)p.out_row[row] : (long)row;
        dst = p.out + orow * p.N + col0;
        if (p.diff_out) {
            // second output: the stored (bf16-rounded) value minus diff_in's row, i.e. what a separate
            // pass over the stored output would compute
            const uint4* x4 = (const uint4*)(p.diff_in + orow * p.N + col0);
            uint4* c4 = (uint4*)(p.diff_out + orow * p.N + col0);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 x = x4[i];
                const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t yb = pack_bf16(v[i * 8 + j * 2], v[i * 8 + j * 2 + 1]);
                    o[j] = pack_bf16(__uint_as_float(yb << 16) - __uint_as_float(xw[j] << 16),
                                     __uint_as_float(yb & 0xffff0000u) - __uint_as_float(xw[j] & 0xffff0000u));
                }
                c4[i] = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    } else {
        // QKV routing: this 32-column chunk lies entirely in q, k or v (C % 32 == 0)
        const int which = col0 / p.C, cc = col0 - which * p.C;
        if (which == 0) dst = p.out + (long)row * p.C + cc;
        else {
            if (kv_base < 0) return;   // cache overflow: flagged when the row map was built
            dst = (which == 1 ? p.k_cache : p.v_cache) + kv_base * p.C + cc;
        }
    }
    uint4* d4 = (uint4*)dst;
#pragma unroll
    for (int i = 0; i < 4; ++i)
        d4[i] = make_uint4(pack_bf16(v[i * 8], v[i * 8 + 1]), pack_bf16(v[i * 8 + 2], v[i * 8 + 3]),
                           pack_bf16(v[i * 8 + 4], v[i * 8 + 5]), pack_bf16(v[i * 8 + 6], v[i * 8 + 7]));
}

template <int BN, int STAGES>
__global__ void __launch_bounds__(kThreads)
gemm_bf16_tn(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
             const GemmParams p)
{
    using L = GemmSmem<BN, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full_bar = (uint64_t*)(smem + STAGES * L::kStageBytes);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* acc_bar = empty_bar + STAGES;
    uint32_t* tmem_slot = (uint32_t*)(acc_bar + 1);
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int num_kb = p.K / BK;
    const int M = true_rows(p);
    if (blockIdx.x == 0 && blockIdx.y == 0) advance_kv_len(p);
    if (m0 >= M) return;            // whole tile past the device-side row count (nothing allocated yet)

    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(acc_bar, 1);
        fence_barrier_init();
        prefetch_tmap(&tmap_a);
        prefetch_tmap(&tmap_w);
    }
    if (warp == 1) tmem_alloc(tmem_slot, BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % STAGES;
                if (kb >= STAGES && !mbar_wait(&empty_bar[s], ((kb / STAGES) - 1) & 1, abort_flag, p.status)) break;
                uint8_t* a_dst = smem + s * L::kStageBytes;
                uint8_t* b_dst = a_dst + L::kABytes;
                mbar_arrive_expect_tx(&full_bar[s], L::kStageBytes);
                tma_load_2d(a_dst, &tmap_a, &full_bar[s], kb * BK, m0);
                tma_load_2d(b_dst, &tmap_w, &full_bar[s], kb * BK, n0);
                issued = kb + 1;
            }
            if (*abort_flag) {
                // let the copies already issued land before the CTA's shared memory is released
                for (int kb = max(0, issued - STAGES); kb < issued; ++kb)
                    mbar_drain(&full_bar[kb % STAGES], (kb / STAGES) & 1);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(BM, BN, 0);
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                const int s = kb % STAGES;
                ok = mbar_wait(&full_bar[s], (kb / STAGES) & 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(smem + s * L::kStageBytes);
                const uint32_t b_addr = a_addr + L::kABytes;
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk) {
                    const uint64_t adesc = smem_desc_sw128(a_addr + kk * 32, 16, 1024);
                    const uint64_t bdesc = smem_desc_sw128(b_addr + kk * 32, 16, 1024);
                    mma_bf16_ss(tmem_acc, adesc, bdesc, idesc, (kb | kk) ? 1u : 0u);
                }
                mma_commit(&empty_bar[s]);   // frees the stage when these MMAs have read it
            }
            if (ok) mma_commit(acc_bar);     // accumulator complete
        }
    } else {
        // epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31
        const int q = warp & 3;
        const int row = m0 + q * 32 + lane;
        if (mbar_wait_warp(acc_bar, 0, abort_flag, p.status)) {
            tc_fence_after();
            const bool row_ok = row < M;
            long res_base = 0;
            long kv_base = -1;
            if (row_ok) {
                if (p.epilogue == NOVA_EPI_BIAS_RES) res_base = (long)(p.res_row ? p.res_row[row] : row) * p.N;
                if (p.epilogue == NOVA_EPI_QKV) kv_base = (long)p.kv_row[row];
            }
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                const int col0 = n0 + c * 32;
                uint32_t acc[32];
                tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), acc);
                tmem_ld_wait();
                if (!row_ok || col0 >= p.N) continue;
                epilogue_chunk(p, row, col0, acc, res_base, kv_base);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_acc, BN);
    }
}

GemmParams make_params(nova_ctx* ctx, const nova_gemm_args& a)
{
    GemmParams p;
    p.bias = a.bias; p.M = a.M; p.N = a.N; p.K = a.K; p.epilogue = a.epilogue; p.out = a.out;
    p.res = a.res; p.res_row = a.res_row; p.C = a.C; p.k_cache = a.k_cache; p.v_cache = a.v_cache;
    p.kv_row = a.kv_row; p.status = ctx->dev_status;
    p.adv_cu_keep = a.adv_cu_keep; p.adv_kv_len = a.adv_kv_len; p.adv_B = a.adv_B; p.adv_Lmax = a.adv_Lmax;
    p.ent = a.ent; p.m_dev = a.m_dev; p.gate = a.gate; p.img_row = a.img_row;
    p.out_row = a.out_row; p.diff_in = a.diff_in; p.diff_out = a.diff_out;
    return p;
}

// ---- CTA-pair kernel ------------------------------------------------------------------------
constexpr int kPairBM = 256;           // rows of one pair tile (128 per CTA)
constexpr int kPairThreads = 320;      // producer warp, MMA warp, eight epilogue warps

template <int BN, int STAGES>
struct PairSmem {
    static constexpr int kABytes = 128 * BK * 2;           // this CTA's 128 rows of A
    static constexpr int kBBytes = (BN / 2) * BK * 2;      // this CTA's half of the W rows
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTotal = STAGES * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// Work list of one launch: entries [0, tiles_full) are whole 256 x BN tiles in column-major tile
// order; the tiles after those, which would otherwise leave most pairs idle in a last partial wave,
// are each split into two 256 x BN/2 halves (entries tiles_full, tiles_full + 1, ...).
struct PairTile {
    int m0;     // first row of the pair tile
    int n0;     // first column
    int bn;     // columns: BN or BN / 2
};
// `span` > 0: tile index = m_tile + tiles_m * n_tile with span = tiles_m (tiles that run at the same
// time share few W rows and sweep all of A); span < 0: index = n_tile + tiles_n * m_tile with
// -span = tiles_n (they sweep all of W and share few A rows). The launcher picks the order whose
// swept operand is the smaller one, so that the larger one is fetched from HBM only once.
template <int BN>
__device__ __forceinline__ PairTile decode_tile(int entry, int span, int tiles_full)
{
    PairTile t;
    int whole = entry, half = -1;
    if (entry >= tiles_full) {
        const int h = entry - tiles_full;
        whole = tiles_full + (h >> 1);
        half = h & 1;
    }
    const int mt = span > 0 ? whole % span : whole / (-span);
    const int nt = span > 0 ? whole / span : whole % (-span);
    t.m0 = mt * kPairBM;
    t.n0 = nt * BN + (half > 0 ? BN / 2 : 0);
    t.bn = half >= 0 ? BN / 2 : BN;
    return t;
}

// Entry of the work list that pair `pair` handles as its `local`-th tile, or -1 past the end.
// group == 0: entries pair, pair + num_pairs, ... (any tile to any pair). group > 0 (entropy
// epilogue, group = tiles along N, N-fastest order): a pair takes whole row blocks, all their `group`
// column tiles in turn, so that the epilogue threads can carry a row's softmax state across them.
__device__ __forceinline__ int pair_entry(int local, int pair, int num_pairs, int num_tiles, int group)
{
    int e;
    if (group == 0) e = pair + local * num_pairs;
    else e = (pair + (local / group) * num_pairs) * group + local % group;
    return e < num_tiles ? e : -1;
}

// ---- entropy epilogue: running softmax-entropy state of one output row ----------------------
// m = reference maximum, s = sum e^{z-m}, u = sum (z-m) e^{z-m} in the log2 domain (m2 = m log2 e),
// the sums as two partial sums per 64-bit register (packed fp32 arithmetic).
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct EntropyState {
    float m, m2;
    uint64_t s2, u2;
    __device__ __forceinline__ void reset()
    {
        m = -INFINITY; m2 = -INFINITY;
        s2 = pack_f32x2(0.f, 0.f);
        u2 = s2;
    }
    // 32 more logits of the row (fp32 accumulators plus bias)
    __device__ __forceinline__ void add_chunk(const uint32_t (&acc)[32], const __nv_bfloat16* bias)
    {
        constexpr float kLog2e = 1.4426950408889634f;
        float z[32];
        if (bias) {
            const uint4* bias4 = (const uint4*)bias;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 b = bias4[i];
                const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    z[i * 8 + j * 2] = __uint_as_float(acc[i * 8 + j * 2]) + __uint_as_float(bw[j] << 16);
                    z[i * 8 + j * 2 + 1] = __uint_as_float(acc[i * 8 + j * 2 + 1]) + __uint_as_float(bw[j] & 0xffff0000u);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) z[i] = __uint_as_float(acc[i]);
        }
        float cm = z[0];
#pragma unroll
        for (int i = 1; i < 32; ++i) cm = fmaxf(cm, z[i]);
        if (cm > m) {
            // raise the reference: both sums scale by f = e^{m - m'}, u also shifts by (m - m') s
            const float shift = (m - cm) * kLog2e;          // -inf the first time: f = 0
            const float f = ex2_approx(shift);
            float s_lo, s_hi, u_lo, u_hi;
            unpack_f32x2(s2, s_lo, s_hi);
            unpack_f32x2(u2, u_lo, u_hi);
            if (m == -INFINITY) { u_lo = u_hi = 0.f; }
            else {
                u_lo = (u_lo + shift * s_lo) * f;
                u_hi = (u_hi + shift * s_hi) * f;
            }
            s2 = pack_f32x2(s_lo * f, s_hi * f);
            u2 = pack_f32x2(u_lo, u_hi);
            m = cm;
            m2 = cm * kLog2e;
        }
        const uint64_t log2e2 = pack_f32x2(kLog2e, kLog2e), neg_m2 = pack_f32x2(-m2, -m2);
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            const uint64_t d2 = fma_f32x2(pack_f32x2(z[i], z[i + 1]), log2e2, neg_m2);
            float d0, d1;
            unpack_f32x2(d2, d0, d1);
            const uint64_t e2 = pack_f32x2(ex2_approx(d0), ex2_approx(d1));
            s2 = add_f32x2(s2, e2);
            u2 = fma_f32x2(d2, e2, u2);
        }
    }
    // H = ln s - u/s (u in log2 units); non-finite inputs give NaN and flag the status word
    __device__ __forceinline__ float finish(unsigned int* status) const
    {
        float s_lo, s_hi, u_lo, u_hi;
        unpack_f32x2(s2, s_lo, s_hi);
        unpack_f32x2(u2, u_lo, u_hi);
        const float s = s_lo + s_hi, u = u_lo + u_hi;
        float h = logf(s) - (u / s) * 0.6931471805599453f;
        if (!(fabsf(m) < INFINITY) || !(fabsf(h) < INFINITY)) {
            h = __int_as_float(0x7fc00000);
            atomicOr(status, NOVA_DEV_NONFINITE);
        } else if (h <= 0.f) {
            h = 0.f;
        }
        return h;
    }
};

// Role layout as in gemm_bf16_tn. Barriers (all in each CTA's shared memory at equal offsets):
//   full[s]       leader's copy is used: one arrival (its own expect_tx) + the bytes of both CTAs
//   empty[s]      each CTA's copy, signalled in both CTAs by the leader's tcgen05.commit
//   acc_full[a]   each CTA's copy, same; a = accumulator buffer of tile parity
//   acc_empty[a]  leader's copy: one arrival per epilogue warp of both CTAs (16)
template <int BN, int STAGES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
gemm_bf16_tn_pair(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                  const __grid_constant__ CUtensorMap tmap_w_half, const GemmParams p, const int span_host,
                  const int tiles_full_host, const int num_tiles_host, const int group)
{
    using L = PairSmem<BN, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full_bar = (uint64_t*)(smem + STAGES * L::kStageBytes);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* acc_full = empty_bar + STAGES;     // 2
    uint64_t* acc_empty = acc_full + 2;          // 2
    uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();     // 0 = leader
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    if (blockIdx.x == 0) advance_kv_len(p);
    const int num_kb = p.K / BK;
    // The work list is the host's, or, when only the device knows the row count, the same plan
    // rebuilt here from that count (every thread computes the same values).
    int M = p.M, span = span_host, tiles_full = tiles_full_host, num_tiles = num_tiles_host;
    if (p.m_dev) {
        M = true_rows(p);
        const int tiles_m = (M + kPairBM - 1) / kPairBM, tiles_n = (p.N + BN - 1) / BN;
        const int tiles = tiles_m * tiles_n;
        const int rem = tiles % num_pairs;
        tiles_full = (group == 0 && rem > 0 && 2 * rem <= num_pairs) ? tiles - rem : tiles;
        num_tiles = tiles_full + 2 * (tiles - tiles_full);
        span = (group != 0 || M >= p.N) ? -tiles_n : tiles_m;
    }
    constexpr uint32_t kTmemCols = 2 * BN;       // two accumulator buffers

    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], 16);
        }
        fence_barrier_init();
        prefetch_tmap(&tmap_a);
        prefetch_tmap(&tmap_w);
        prefetch_tmap(&tmap_w_half);
    }
    if (warp == 1) tmem_alloc_pair(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                          // both CTAs' barriers exist before either signals the other
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            long it = 0;                         // k-blocks issued so far over all tiles of this pair
            bool ok = true;
            for (int local = 0; ok; ++local) {
                const int tile = pair_entry(local, pair, num_pairs, num_tiles, group);
                if (tile < 0) break;
                const PairTile t = decode_tile<BN>(tile, span, tiles_full);
                const int m0 = t.m0 + (int)rank * 128;
                const int n0 = t.n0 + (int)rank * (t.bn / 2);
                const CUtensorMap* wmap = (t.bn == BN) ? &tmap_w : &tmap_w_half;
                const uint32_t stage_tx = 2u * (uint32_t)(L::kABytes + (t.bn / 2) * BK * 2);
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = (int)(it % STAGES);
                    if (it >= STAGES && !mbar_wait(&empty_bar[s], (uint32_t)((it / STAGES) - 1) & 1, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    uint8_t* a_dst = smem + s * L::kStageBytes;
                    uint8_t* b_dst = a_dst + L::kABytes;
                    if (rank == 0) mbar_arrive_expect_tx(&full_bar[s], stage_tx);
                    const uint32_t bar = map_to_cta(smem_u32(&full_bar[s]), 0);
                    tma_load_2d_pair(a_dst, &tmap_a, bar, kb * BK, m0);
                    tma_load_2d_pair(b_dst, wmap, bar, kb * BK, n0);
                }
            }
            if (*abort_flag && rank == 0) {
                // let the copies already issued land before shared memory is released
                for (long k2 = (it > STAGES ? it - STAGES : 0); k2 < it; ++k2)
                    mbar_drain(&full_bar[k2 % STAGES], (uint32_t)(k2 / STAGES) & 1);
            }
        }
    } else if (warp == 1) {
        if (rank == 0 && lane == 0) {
            // One elected thread of the leader CTA does nothing but wait and issue. Per 64-wide k-block
            // the tensor core works 512 clocks (four M=256, N=256, K=16 instructions); the thread spends
            // about 80 clocks per instruction, 50 on the commit and 65 on a wait that is already
            // satisfied, which leaves a margin. The earlier form, the whole warp in lockstep with every
            // lane polling the barrier and a vote after it, paid about 300 clocks per wait and made the
            // issuing warp, not the tensor core, the limit of the main loop (tensor pipe 75 % active).
            constexpr uint32_t idesc_whole = idesc_bf16_f32(kPairBM, BN, 0);
            constexpr uint32_t idesc_half = idesc_bf16_f32(kPairBM, BN / 2, 0);
            const uint64_t a_desc = smem_desc_sw128(smem_u32(smem), 16, 1024);
            int s = 0;                 // ring position and phase parity of the next k-block
            uint32_t par = 0;
            int local = 0;
            bool ok = true;
            for (; ok; ++local) {
                const int tile = pair_entry(local, pair, num_pairs, num_tiles, group);
                if (tile < 0) break;
                const int a = local & 1;
                if (local >= 2) {
                    ok = mbar_wait(&acc_empty[a], (uint32_t)((local >> 1) - 1) & 1, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                }
                const uint32_t d_tmem = tmem_base + (uint32_t)(a * BN);
                const uint32_t idesc = (tile < tiles_full) ? idesc_whole : idesc_half;
                for (int kb = 0; kb < num_kb; ++kb) {
                    ok = mbar_wait(&full_bar[s], par, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t ad = a_desc + (uint32_t)s * (uint32_t)(L::kStageBytes >> 4);
                    const uint64_t bd = ad + (uint32_t)(L::kABytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)
                        mma_bf16_ss_pair(d_tmem, ad + (uint32_t)(kk * 2), bd + (uint32_t)(kk * 2), idesc, (kb | kk) ? 1u : 0u);
                    mma_commit_pair(&empty_bar[s], 3);      // frees the stage in both CTAs
                    if (++s == STAGES) { s = 0; par ^= 1u; }
                }
                if (ok) mma_commit_pair(&acc_full[a], 3);    // accumulator complete in both CTAs
            }
        }
    } else {
        // epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31 of this CTA's half of the tile. Two
        // warps share each lane quarter and take alternate 32-column chunks: the epilogue of a tile
        // is a long chain of dependent instructions per thread, and with one warp per quarter the
        // GELU epilogue took longer than the tile's main loop. (The entropy epilogue carries a row's
        // state from chunk to chunk in one thread, so there the second warp of a quarter only
        // signals.)
        const int q = warp & 3;
        const bool entropy_epi = (p.epilogue == NOVA_EPI_ENTROPY);
        const int c_first = entropy_epi ? 0 : ((warp - 2) >> 2), c_step = entropy_epi ? 1 : 2;
        const bool idle_warp = entropy_epi && warp >= 6;
        const uint32_t acc_empty_leader = map_to_cta(smem_u32(&acc_empty[0]), 0);
        int local = 0;
        bool ok = true;
        EntropyState est;
        est.reset();
        for (; ok; ++local) {
            const int tile = pair_entry(local, pair, num_pairs, num_tiles, group);
            if (tile < 0) break;
            const int a = local & 1;
            const PairTile t = decode_tile<BN>(tile, span, tiles_full);
            const int row = t.m0 + (int)rank * 128 + q * 32 + lane;
            const int n0 = t.n0, n_chunks = t.bn / 32;
            ok = mbar_wait_warp(&acc_full[a], (uint32_t)(local >> 1) & 1, abort_flag, p.status);
            if (!ok) break;
            tc_fence_after();
            const bool row_ok = row < M;
            long res_base = 0;
            long kv_base = -1;
            if (row_ok) {
                if (p.epilogue == NOVA_EPI_BIAS_RES) res_base = (long)(p.res_row ? p.res_row[row] : row) * p.N;
                if (p.epilogue == NOVA_EPI_QKV) kv_base = (long)p.kv_row[row];
            }
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * BN);
#pragma unroll 1
            for (int c = c_first; c < n_chunks && !idle_warp; c += c_step) {
                const int col0 = n0 + c * 32;
                uint32_t acc[32];
                tmem_ld32(t_addr + (uint32_t)(c * 32), acc);
                tmem_ld_wait();
                if (!row_ok || col0 >= p.N) continue;
                if (p.epilogue == NOVA_EPI_ENTROPY) est.add_chunk(acc, p.bias ? p.bias + col0 : nullptr);
                else epilogue_chunk(p, row, col0, acc, res_base, kv_base);
            }
            if (p.epilogue == NOVA_EPI_ENTROPY && !idle_warp && t.n0 + BN >= p.N) {
                // last column tile of this row block: the row's entropy is complete
                if (row_ok) p.ent[row] = est.finish(p.status);
                est.reset();
            }
            // this warp has read its part of the buffer: tell the leader's MMA thread
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_leader + (uint32_t)(a * 8));
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();     // the peer may still read this CTA's shared memory or signal its barriers
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

template <int BN, int STAGES>
nova_status launch_pair(nova_ctx* ctx, const nova_gemm_args& a, cudaStream_t st)
{
    using L = PairSmem<BN, STAGES>;
    CUtensorMap ta, tw;
    const uint64_t da[2] = {(uint64_t)a.K, (uint64_t)a.M}, sa[1] = {(uint64_t)a.K * 2};
    const uint64_t dw[2] = {(uint64_t)a.K, (uint64_t)a.N}, sw[1] = {(uint64_t)a.K * 2};
    CUtensorMap tw_half;
    if (!make_tmap_bf16(ctx, &ta, a.A, 2, da, sa, 128) || !make_tmap_bf16(ctx, &tw, a.W, 2, dw, sw, BN / 2) ||
        !make_tmap_bf16(ctx, &tw_half, a.W, 2, dw, sw, BN / 4))
        return nova_fail(ctx, NOVA_ERR_CUDA, "gemm: cuTensorMapEncodeTiled failed");
    auto kern = gemm_bf16_tn_pair<BN, STAGES>;
    static bool attr_done[64];
    if (ctx->device < 64 && !attr_done[ctx->device]) {
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal));
        attr_done[ctx->device] = true;
    }
    GemmParams p = make_params(ctx, a);
    const int tiles_m = (a.M + kPairBM - 1) / kPairBM, tiles_n = (a.N + BN - 1) / BN;
    const int tiles = tiles_m * tiles_n;
    const bool entropy = (a.epilogue == NOVA_EPI_ENTROPY);
    // the entropy epilogue hands whole row blocks to pairs; otherwise any tile goes to any pair
    const int pairs = min(entropy ? tiles_m : tiles, ctx->num_sms / 2);
    // a last partial wave that would occupy at most half of the pairs runs as half-width tiles
    const int rem = tiles % pairs;
    const int tiles_full = (!entropy && rem > 0 && 2 * rem <= pairs) ? tiles - rem : tiles;
    const int entries = tiles_full + 2 * (tiles - tiles_full);
    {
        nova_launch_scope scope(ctx, a.cat, st);
        // sweep the smaller operand; the entropy epilogue needs the N-fastest order
        const int span = (entropy || (long)a.M >= (long)a.N) ? -tiles_n : tiles_m;
        kern<<<dim3(2 * pairs), kPairThreads, L::kTotal, st>>>(ta, tw, tw_half, p, span, tiles_full, entries,
                                                           entropy ? tiles_n : 0);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

template <int BN, int STAGES>
nova_status launch(nova_ctx* ctx, const nova_gemm_args& a, cudaStream_t st)
{
    using L = GemmSmem<BN, STAGES>;
    CUtensorMap ta, tw;
    const uint64_t da[2] = {(uint64_t)a.K, (uint64_t)a.M}, sa[1] = {(uint64_t)a.K * 2};
    const uint64_t dw[2] = {(uint64_t)a.K, (uint64_t)a.N}, sw[1] = {(uint64_t)a.K * 2};
    if (!make_tmap_bf16(ctx, &ta, a.A, 2, da, sa, BM) || !make_tmap_bf16(ctx, &tw, a.W, 2, dw, sw, BN))
        return nova_fail(ctx, NOVA_ERR_CUDA, "gemm: cuTensorMapEncodeTiled failed");
    auto kern = gemm_bf16_tn<BN, STAGES>;
    if (!ctx->attr_gemm) {
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal));
        ctx->attr_gemm = true;
    }
    GemmParams p = make_params(ctx, a);
    dim3 grid((a.N + BN - 1) / BN, (a.M + BM - 1) / BM);
    {
        nova_launch_scope scope(ctx, a.cat, st);
        kern<<<grid, kThreads, L::kTotal, st>>>(ta, tw, p);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

}  // namespace

nova_status nova_launch_gemm(nova_ctx* ctx, const nova_gemm_args& a, cudaStream_t st)
{
    if (a.M <= 0) return NOVA_OK;
    if (a.K % BK || a.N % 32 || a.K < BK) return nova_fail(ctx, NOVA_ERR_SHAPE, "gemm: K must be a multiple of 64 and N of 32");
    // CTA pairs with 256 x 256 tiles once there is at least one tile per pair of SMs; below that the
    // single-CTA 128 x 128 tiles spread a small problem over more SMs.
    const long tiles_pair = (long)((a.M + 255) / 256) * ((a.N + 255) / 256);
    if (a.epilogue == NOVA_EPI_ENTROPY) {
        if (ctx->num_sms < 2) return nova_fail(ctx, NOVA_ERR_SHAPE, "gemm: the entropy epilogue needs the CTA-pair kernel");
        return launch_pair<256, 6>(ctx, a, st);
    }
    if (tiles_pair >= ctx->num_sms / 2 && ctx->num_sms >= 2) return launch_pair<256, 6>(ctx, a, st);
    return launch<128, 3>(ctx, a, st);
}

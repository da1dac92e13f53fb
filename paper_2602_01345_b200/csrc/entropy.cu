// Eq. 4 / Eq. 7: per-token softmax entropy over the codebook logits and its per-image mean.
//
// One warp owns one row. The row is pulled from HBM exactly once and held packed in registers;
// the warp takes the row maximum m, then one pass gives
//   s = sum e^{z-m},  u = sum (z-m) e^{z-m},  H = ln s - u / s,
// two logits per instruction (packed fp32). Rows of 2, 4 or 8 KiB (V = 4096 bf16 is 8 KiB) are
// staged through a shared-memory ring by bulk copies in a persistent kernel that also takes the
// per-image means; other shapes use one-warp-per-row kernels and a separate mean kernel.
#include "tc_common.cuh"

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void unpack_bf16x2(uint32_t w, float& lo, float& hi)
{
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xffff0000u);
}

// finishing step shared by all kernels: lane 0 writes the row result
__device__ __forceinline__ float finish_row(float m, float s, float u, float* ent, long row,
                                            unsigned int* status)
{
    // H = ln s - u/s with u accumulated in the log2 domain: d2 = (z-m)*log2e, u2 = sum d2 * 2^d2
    float h = logf(s) - (u / s) * kLn2;   // precise log once per row: ln 1 must be exactly 0
    if (!(m < INFINITY) || !(m > -INFINITY) || !(s > 0.f) || h != h) {
        h = __int_as_float(0x7fc00000);
        atomicOr(status, NOVA_DEV_NONFINITE);
    } else if (h <= 0.f) {
        h = 0.f;   // also turns -0 into +0; true entropy is never negative
    }
    ent[row] = h;
    return h;
}

// ---- two fp32 values per 64-bit register: one instruction does both lanes' arithmetic ----------
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

// Exact two-pass evaluation of one row straight from global memory (the row is in L2): used for
// rows that do not fit the register kernels and for the rare rows whose fast result is not
// finite. -inf logits contribute 0; NaN or +inf logits leave m or s non-finite, which finish_row
// reports. All 32 lanes of the warp call it together; every lane gets the row's m, s, u.
template <bool BF16>
__device__ __forceinline__ void entropy_row_exact(const char* base, int V, int lane, float& m, float& s, float& u)
{
    auto at = [&](int e) -> float {
        return BF16 ? __bfloat162float(((const __nv_bfloat16*)base)[e]) : ((const float*)base)[e];
    };
    float mm = -INFINITY;
    bool nan = false;
    for (int e = lane; e < V; e += 32) {
        const float z = at(e);
        nan |= (z != z);
        mm = fmaxf(mm, z);
    }
    mm = warp_max(mm);
    float ss = 0.f, uu = 0.f;
    for (int e = lane; e < V; e += 32) {
        const float d = (at(e) - mm) * kLog2e;
        const float ex = fast_exp2(d);
        ss += ex;
        uu = fmaf(d == -INFINITY ? 0.f : d, ex, uu);
    }
    if (nan) ss = __int_as_float(0x7fc00000);
    m = mm;
    s = warp_sum(ss);
    u = warp_sum(uu);
}

// Entropy sums of one row held as VEC packed 16-byte vectors per lane (BF16: 8 logits per vector,
// F32: 4). First the row maximum m (packed bf16 maxima, then one warp reduction), then one
// branch-free pass with, per pair of logits, two unpacks, one packed multiply-add
// d = z * log2(e) - m * log2(e), two ex2, one packed add into s and one packed multiply-add into u
// (u in the log2 domain), spread over independent accumulators. This pass handles finite logits
// only: a -inf logit gives -inf * 0 = NaN in u, a NaN or +inf logit poisons m or s; any row whose
// result is not finite is recomputed by entropy_row_exact, which treats every special value as
// documented. On return every lane holds the row's m, s, u.
template <int VEC, bool BF16>
__device__ __forceinline__ void entropy_row_from_regs(const uint4 (&reg)[VEC], const char* base, int V, int lane,
                                                      float& m_out, float& s_out, float& u_out)
{
    float m;
    if (BF16) {
        __nv_bfloat162 mx[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) mx[q] = *reinterpret_cast<const __nv_bfloat162*>(&(&reg[0].x)[q]);
#pragma unroll
        for (int i = 1; i < VEC; ++i) {
            const uint32_t w[4] = {reg[i].x, reg[i].y, reg[i].z, reg[i].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) mx[q] = __hmax2(mx[q], *reinterpret_cast<const __nv_bfloat162*>(&w[q]));
        }
        const __nv_bfloat162 t = __hmax2(__hmax2(mx[0], mx[1]), __hmax2(mx[2], mx[3]));
        float lo, hi;
        unpack_bf16x2(*reinterpret_cast<const uint32_t*>(&t), lo, hi);
        m = fmaxf(lo, hi);
    } else {
        float mx[4] = {__uint_as_float(reg[0].x), __uint_as_float(reg[0].y), __uint_as_float(reg[0].z), __uint_as_float(reg[0].w)};
#pragma unroll
        for (int i = 1; i < VEC; ++i) {
            mx[0] = fmaxf(mx[0], __uint_as_float(reg[i].x));
            mx[1] = fmaxf(mx[1], __uint_as_float(reg[i].y));
            mx[2] = fmaxf(mx[2], __uint_as_float(reg[i].z));
            mx[3] = fmaxf(mx[3], __uint_as_float(reg[i].w));
        }
        m = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
    }
    m = warp_max(m);

    const uint64_t log2e2 = pack_f32x2(kLog2e, kLog2e);
    const uint64_t neg_m2 = pack_f32x2(-m * kLog2e, -m * kLog2e);
    uint64_t s2[4], u2[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) s2[a] = u2[a] = pack_f32x2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const uint32_t w[4] = {reg[i].x, reg[i].y, reg[i].z, reg[i].w};
        if (BF16) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float lo, hi;
                unpack_bf16x2(w[q], lo, hi);
                const uint64_t d2 = fma_f32x2(pack_f32x2(lo, hi), log2e2, neg_m2);
                float d0, d1;
                unpack_f32x2(d2, d0, d1);
                const uint64_t e2 = pack_f32x2(fast_exp2(d0), fast_exp2(d1));
                s2[q] = add_f32x2(s2[q], e2);
                u2[q] = fma_f32x2(d2, e2, u2[q]);
            }
        } else {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const uint64_t d2 = fma_f32x2(pack_f32x2(__uint_as_float(w[2 * q]), __uint_as_float(w[2 * q + 1])), log2e2, neg_m2);
                float d0, d1;
                unpack_f32x2(d2, d0, d1);
                const uint64_t e2 = pack_f32x2(fast_exp2(d0), fast_exp2(d1));
                s2[2 * (i & 1) + q] = add_f32x2(s2[2 * (i & 1) + q], e2);
                u2[2 * (i & 1) + q] = fma_f32x2(d2, e2, u2[2 * (i & 1) + q]);
            }
        }
    }
    const uint64_t st = add_f32x2(add_f32x2(s2[0], s2[1]), add_f32x2(s2[2], s2[3]));
    const uint64_t ut = add_f32x2(add_f32x2(u2[0], u2[1]), add_f32x2(u2[2], u2[3]));
    float s_lo, s_hi, u_lo, u_hi;
    unpack_f32x2(st, s_lo, s_hi);
    unpack_f32x2(ut, u_lo, u_hi);
    float s = warp_sum(s_lo + s_hi);
    float u = warp_sum(u_lo + u_hi);
    const float h = logf(s) - (u / s) * kLn2;
    // Anything unusual (-inf, +inf or NaN logits) shows up as a non-finite result and takes the
    // exact path; the decision is the same in every lane.
    if (!(fabsf(h) < INFINITY)) entropy_row_exact<BF16>(base, V, lane, m, s, u);
    m_out = m; s_out = s; u_out = u;
}

// One warp per row, the row loaded straight into registers: all loads of the row are issued before
// the first use (VEC * 16 bytes in flight per lane).
template <int VEC, bool BF16>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
entropy_rows_reg(const void* __restrict__ logits, long rows, int V, long row_stride,
                 float* __restrict__ ent, unsigned int* status)
{
    constexpr int PER = BF16 ? 8 : 4;
    const int lane = threadIdx.x & 31;
    const long row = (long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int n_vec = V / PER;
    const char* base = (const char*)logits + row * row_stride * (BF16 ? 2 : 4);
    const uint4* src = (const uint4*)base;

    float m, s, u;
    if (n_vec * PER != V || n_vec != VEC * 32) {
        // the row does not fill the register tile exactly (same for every row of the launch)
        entropy_row_exact<BF16>(base, V, lane, m, s, u);
    } else {
        uint4 reg[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) reg[i] = ld_stream(src + i * 32 + lane);
        entropy_row_from_regs<VEC, BF16>(reg, base, V, lane, m, s, u);
    }
    if (lane == 0) finish_row(m, s, u, ent, row, status);
}

// ---- persistent kernel: rows staged through a shared-memory ring by bulk copies ----------------
// One CTA per SM. A producer thread keeps the ring's slots (whole rows, 128 KB) in flight with
// cp.async.bulk, one copy per row, completion counted on an mbarrier; sixteen consumer warps take
// rows from the ring in turn, move the row into registers, hand the slot back at once and then do
// the arithmetic. HBM sees one deep, steady stream per SM instead of waves of CTAs that load, then
// compute. The per-segment means are completed by whichever CTA arrives last at a fixed-point
// accumulator in global memory; integer addition commutes, so the result does not depend on the order.
// Row i of a CTA goes to slot i % kSlots and to consumer warp i % 16; kSlots is a multiple of 16, so
// every use of a slot is consumed by the same warp, in order. That matters: a parity wait for use
// n of a slot succeeds at once while use n-1 has not completed yet, and bulk copies may land out of
// order (a copy that misses the TLB can trail later ones by microseconds), so a warp must never
// poll a slot whose previous use some other warp has yet to see.
constexpr int kRingConsumers = 16;
constexpr int kRingProducers = 4;
constexpr int kRingThreads = (kRingConsumers + 1) * 32;
constexpr int kMaxMeanSegments = NOVA_MEAN_MAX_SEGMENTS;
constexpr int kRingBytes = 128 * 1024;

// Bulk copy global -> shared of `bytes` (multiple of 16, both addresses 16-byte aligned).
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(tc::smem_u32(dst)), "l"(src), "r"(bytes), "r"(tc::smem_u32(bar)) : "memory");
}

// Logits of several layers in one launch: layer l's [S, N, V] tensor starts at p[l]; row r of the
// launch is row r % rows_per_layer of layer r / rows_per_layer.
constexpr int kMaxEntropyLayers = 64;
struct LayerPtrs {
    const char* p[kMaxEntropyLayers];
};

template <int VEC, bool BF16>
__global__ void __launch_bounds__(kRingThreads, 1)
entropy_rows_ring(const LayerPtrs layers, long rows_per_layer, long rows, int V, long row_stride_bytes,
                  float* __restrict__ ent, float* __restrict__ mean, int seg_rows, int n_seg,
                  unsigned int* status, unsigned long long* __restrict__ accum, int fix_shift)
{
    // row counts fit 31 bits (checked by the launcher): 32-bit division, not the much slower 64-bit one
    const unsigned int rpl = (unsigned int)rows_per_layer;
    auto row_ptr = [&](long row) -> const char* {
        const unsigned int l = (unsigned int)row / rpl;
        return layers.p[l] + (long)((unsigned int)row - l * rpl) * row_stride_bytes;
    };
    using namespace tc;
    constexpr int kRowBytes = VEC * 512;
    constexpr int kSlots = kRingBytes / kRowBytes;
    static_assert(kSlots % kRingConsumers == 0, "each slot must belong to one consumer warp");
    static_assert(kSlots % kRingProducers == 0, "each slot must belong to one producer lane");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* ring = (uint8_t*)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    uint64_t* full_bar = (uint64_t*)(ring + kSlots * kRowBytes);
    uint64_t* empty_bar = full_bar + kSlots;
    float* warp_part = (float*)(empty_bar + kSlots);       // [kRingConsumers][n_seg] partial sums per warp
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long G = gridDim.x;
    const long n_my = (rows > blockIdx.x) ? (rows - blockIdx.x + G - 1) / G : 0;   // rows b, b+G, ...

    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        for (int i = 0; i < kSlots; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], 1);
        }
        fence_barrier_init();
    }
    if (mean)
        for (int i = threadIdx.x; i < kRingConsumers * n_seg; i += kRingThreads) warp_part[i] = 0.f;
    __syncthreads();

    if (warp == kRingConsumers) {
        // kRingProducers lanes issue the copies, lane p those of rows p, p + kRingProducers, ... of the
        // CTA (slots p, p + kRingProducers, ... : kSlots is a multiple of kRingProducers). A row must
        // be issued every ~190 clocks to keep up with HBM, and one thread's wait on the slot, its
        // expect_tx and the copy instruction take about that long.
        if (lane < kRingProducers) {
            long issued = -1;          // last row index this lane issued
            for (long i = lane; i < n_my; i += kRingProducers) {
                const int slot = (int)(i % kSlots);
                if (i >= kSlots && !mbar_wait(&empty_bar[slot], (uint32_t)((i / kSlots) - 1) & 1, abort_flag, status)) break;
                const long row = blockIdx.x + i * G;
                mbar_arrive_expect_tx(&full_bar[slot], kRowBytes);
                bulk_load(ring + slot * kRowBytes, row_ptr(row), kRowBytes, &full_bar[slot]);
                issued = i;
            }
            if (*abort_flag)
                for (long i = issued; i >= 0 && i > issued - kSlots; i -= kRingProducers)
                    mbar_drain(&full_bar[i % kSlots], (uint32_t)(i / kSlots) & 1);
        }
    } else {
        // running sum of this warp's entropies in the segment it is in (rows come in rising order)
        int cur_seg = -1;
        float seg_acc = 0.f;
        for (long i = warp; i < n_my; i += kRingConsumers) {
            const int slot = (int)(i % kSlots);
            if (!mbar_wait_warp(&full_bar[slot], (uint32_t)(i / kSlots) & 1, abort_flag, status)) break;
            const uint4* src = (const uint4*)(ring + slot * kRowBytes);
            uint4 reg[VEC];
#pragma unroll
            for (int v = 0; v < VEC; ++v) reg[v] = src[v * 32 + lane];
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[slot]);       // the row now lives in registers
            const long row = blockIdx.x + i * G;
            float m, s_sum, u;
            entropy_row_from_regs<VEC, BF16>(reg, row_ptr(row), V, lane, m, s_sum, u);
            if (lane == 0) {
                const float h = finish_row(m, s_sum, u, ent, row, status);
                if (mean) {
                    const int seg = (int)((unsigned int)row / (unsigned int)seg_rows);   // rows < 2^31 (checked by the launcher)
                    if (seg != cur_seg) {
                        if (cur_seg >= 0) warp_part[warp * n_seg + cur_seg] = seg_acc;
                        cur_seg = seg;
                        seg_acc = 0.f;
                    }
                    seg_acc += h;
                }
            }
        }
        if (lane == 0 && mean && cur_seg >= 0) warp_part[warp * n_seg + cur_seg] = seg_acc;
    }
    if (!mean) return;

    // ---- means ---------------------------------------------------------------------------------
    // A CTA's partial sum of a segment is added in a fixed order (a warp's rows in row order, the 16
    // warps in warp order) and then joins the other CTAs' in ONE 64-bit atomic add per segment:
    //   bits 63..56  CTAs that have arrived      bits 55..46  how many of them had a non-finite sum
    //   bits 45..0   sum of the partial sums in fixed point (2^-fix_shift units)
    // Integer addition commutes, so the total does not depend on the order of arrival, and the add
    // that completes the count returns everything needed: that thread writes the mean and clears
    // the accumulator for the next launch. No fence, no second pass over partial results.
    __syncthreads();
    for (int sg = threadIdx.x; sg < n_seg; sg += kRingThreads) {
        float acc = 0.f;
        for (int w = 0; w < kRingConsumers; ++w) acc += warp_part[w * n_seg + sg];
        const bool finite = (acc >= 0.f) && (acc < INFINITY);
        unsigned long long add = 1ull << 56;
        if (finite) add += (unsigned long long)__float2ll_rn(ldexpf(acc, fix_shift));
        else add += 1ull << 46;
        const unsigned long long old = atomicAdd(&accum[sg], add);
        if ((old >> 56) == gridDim.x - 1) {
            const unsigned long long tot = old + add;
            const double sum = (double)(tot & ((1ull << 46) - 1)) * exp2(-(double)fix_shift);
            mean[sg] = ((tot >> 46) & 0x3ffull) ? __int_as_float(0x7fc00000) : (float)(sum / (double)seg_rows);
            accum[sg] = 0ull;
        }
    }
}

// Any V: two reads of the row (the second one is served by L1/L2).
template <bool BF16>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
entropy_rows_stream(const void* __restrict__ logits, long rows, int V, long row_stride,
                    float* __restrict__ ent, unsigned int* status)
{
    const int lane = threadIdx.x & 31;
    const long row = (long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (row >= rows) return;
    const char* base = (const char*)logits + row * row_stride * (BF16 ? 2 : 4);
    float m, s, u;
    entropy_row_exact<BF16>(base, V, lane, m, s, u);
    if (lane == 0) finish_row(m, s, u, ent, row, status);
}

// mean[s] = (1/N) sum_i ent[s, i]; one block per segment, fixed summation tree.
__global__ void __launch_bounds__(1024) entropy_mean(const float* __restrict__ ent, int N,
                                                    float* __restrict__ mean)
{
    __shared__ float part[32];
    const float* e = ent + (long)blockIdx.x * N;
    float acc = 0.f;
    for (int i = threadIdx.x; i < N; i += blockDim.x) acc += e[i];
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x < 32) {
        float v = (threadIdx.x < (blockDim.x >> 5)) ? part[threadIdx.x] : 0.f;
        v = warp_sum(v);
        if (threadIdx.x == 0) mean[blockIdx.x] = v / (float)N;
    }
}

template <bool BF16>
void launch_rows(const void* logits, long rows, int V, long row_stride, float* ent,
                 unsigned int* status, cudaStream_t st)
{
    constexpr int PER = BF16 ? 8 : 4;
    const int n_vec = V / PER;
    const int vec_per_lane = (n_vec + 31) / 32;
    const unsigned blocks = (unsigned)((rows + kWarpsPerBlock - 1) / kWarpsPerBlock);
    const dim3 grid(blocks), block(kWarpsPerBlock * 32);
#define NOVA_ENT_CASE(VEC)                                                                     \
    entropy_rows_reg<VEC, BF16><<<grid, block, 0, st>>>(logits, rows, V, row_stride, ent, status)
    if (vec_per_lane <= 1) NOVA_ENT_CASE(1);
    else if (vec_per_lane <= 2) NOVA_ENT_CASE(2);
    else if (vec_per_lane <= 4) NOVA_ENT_CASE(4);
    else if (vec_per_lane <= 8) NOVA_ENT_CASE(8);
    else if (vec_per_lane <= 16) NOVA_ENT_CASE(16);
    else if (vec_per_lane <= 32 && !BF16) NOVA_ENT_CASE(32);
    else entropy_rows_stream<BF16><<<grid, block, 0, st>>>(logits, rows, V, row_stride, ent, status);
#undef NOVA_ENT_CASE
}

template <int VEC, bool BF16>
nova_status launch_ring(nova_ctx* ctx, const LayerPtrs& layers, long rows_per_layer, long rows, int V, long stride_bytes,
                        float* ent, float* mean, int N, int S, cudaStream_t st)
{
    constexpr int kSlots = kRingBytes / (VEC * 512);
    const size_t smem = kRingBytes + 128 + 2 * sizeof(uint64_t) * kSlots + sizeof(float) * kRingConsumers * kMaxMeanSegments;
    static bool attr_done[64];
    if (ctx->device < 64 && !attr_done[ctx->device]) {
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(entropy_rows_ring<VEC, BF16>,
                                                  cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_done[ctx->device] = true;
    }
    const int grid = (int)(rows < ctx->num_sms ? rows : ctx->num_sms);
    // fixed-point scale of the mean accumulators: a segment's sum is below N * ln(V) <= 24 N, and
    // has to stay below 2^46
    int fix_shift = 30;
    while (fix_shift > 0 && 24.0 * (double)N * exp2((double)fix_shift) >= 70368744177664.0 /* 2^46 */) --fix_shift;
    entropy_rows_ring<VEC, BF16><<<grid, kRingThreads, smem, st>>>(
        layers, rows_per_layer, rows, V, stride_bytes, ent, mean, N, S, ctx->dev_status,
        (unsigned long long*)(ctx->dev_status + NOVA_STATUS_WORDS), fix_shift);
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

}  // namespace

// Entropy of n_layers tensors [S, N, V] (one per layer of a scale; `layers` holds their device
// addresses) into ent [n_layers, S, N] and mean [n_layers, S]: one launch of the persistent ring
// kernel over all n_layers * S * N rows where the shape allows it, else one launch per layer.
static nova_status entropy_layers(nova_ctx* ctx, const void* const* layers, int n_layers, nova_dtype dt,
                                  int S, int N, int V, int64_t row_stride, float* ent, float* mean, void* stream,
                                  const char* who)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (n_layers < 0 || S < 0 || N < 0 || V < 1 || (dt != NOVA_BF16 && dt != NOVA_F32))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_scale_entropy: bad layer count, S, N, V or dtype");
    const long rows_per_layer = (long)S * N;
    const long rows = rows_per_layer * n_layers;
    if (rows == 0) return NOVA_OK;
    if (!layers || !ent) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_scale_entropy: null pointer");
    const int per = (dt == NOVA_BF16) ? 8 : 4;
    for (int l = 0; l < n_layers; ++l) {
        if (!layers[l]) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_scale_entropy: null pointer");
        if (row_stride < V || (row_stride % per) != 0 || !nova_aligned16(layers[l]))
            return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_scale_entropy: logits rows must start on 16-byte boundaries");
    }
    NOVA_DEVICE_GUARD(ctx, who);
    cudaStream_t st = (cudaStream_t)stream;
    const int elt = (dt == NOVA_BF16) ? 2 : 4;
    const long row_bytes = (long)V * elt;
    const long segs = (long)n_layers * S;
    if ((row_bytes == 2048 || row_bytes == 4096 || row_bytes == 8192) && rows >= 64 && rows <= 0x7fffffffL &&
        n_layers <= kMaxEntropyLayers &&
        (!mean || (segs <= NOVA_MEAN_MAX_SEGMENTS && ctx->num_sms <= NOVA_MEAN_MAX_CTAS))) {
        // persistent ring kernel over the rows of all layers
        LayerPtrs lp;
        memset(&lp, 0, sizeof(lp));
        for (int l = 0; l < n_layers; ++l) lp.p[l] = (const char*)layers[l];
        const long stride_bytes = (long)row_stride * elt;
        nova_launch_scope scope(ctx, NOVA_K_ENTROPY, st);
        const bool bf = (dt == NOVA_BF16);
        const int sg = (int)segs;
        if (row_bytes == 2048) return bf ? launch_ring<4, true>(ctx, lp, rows_per_layer, rows, V, stride_bytes, ent, mean, N, sg, st)
                                         : launch_ring<4, false>(ctx, lp, rows_per_layer, rows, V, stride_bytes, ent, mean, N, sg, st);
        if (row_bytes == 4096) return bf ? launch_ring<8, true>(ctx, lp, rows_per_layer, rows, V, stride_bytes, ent, mean, N, sg, st)
                                         : launch_ring<8, false>(ctx, lp, rows_per_layer, rows, V, stride_bytes, ent, mean, N, sg, st);
        return bf ? launch_ring<16, true>(ctx, lp, rows_per_layer, rows, V, stride_bytes, ent, mean, N, sg, st)
                  : launch_ring<16, false>(ctx, lp, rows_per_layer, rows, V, stride_bytes, ent, mean, N, sg, st);
    }
    if (n_layers > 1) {
        // shapes the ring kernel does not take: layer by layer
        for (int l = 0; l < n_layers; ++l) {
            const nova_status rc = entropy_layers(ctx, layers + l, 1, dt, S, N, V, row_stride, ent + (long)l * rows_per_layer,
                                                  mean ? mean + (long)l * S : nullptr, stream, who);
            if (rc != NOVA_OK) return rc;
        }
        return NOVA_OK;
    }
    {
        nova_launch_scope scope(ctx, NOVA_K_ENTROPY, st);
        if (dt == NOVA_BF16) launch_rows<true>(layers[0], rows, V, row_stride, ent, ctx->dev_status, st);
        else launch_rows<false>(layers[0], rows, V, row_stride, ent, ctx->dev_status, st);
    }
    if (mean) {
        nova_launch_scope scope(ctx, NOVA_K_ENTROPY_MEAN, st);
        entropy_mean<<<S, 1024, 0, st>>>(ent, N, mean);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

extern "C" nova_status nova_scale_entropy(nova_ctx* ctx, const void* logits, nova_dtype dt,
                                          int S, int N, int V, int64_t row_stride,
                                          float* ent, float* mean, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if ((long)S * N != 0 && !logits) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_scale_entropy: null pointer");
    return entropy_layers(ctx, &logits, 1, dt, S, N, V, row_stride, ent, mean, stream, "nova_scale_entropy");
}

extern "C" nova_status nova_scale_entropy_layers(nova_ctx* ctx, const void* const* logits, int n_layers, nova_dtype dt,
                                                 int S, int N, int V, int64_t row_stride,
                                                 float* ent, float* mean, void* stream)
{
    return entropy_layers(ctx, logits, n_layers, dt, S, N, V, row_stride, ent, mean, stream, "nova_scale_entropy_layers");
}

// Eq. 4 / Eq. 7 one step earlier: entropy of softmax(x W^T + b) without the logits ever reaching
// HBM. The head GEMM runs on the tensor cores (CTA-pair kernel) and its epilogue threads, one row
// each, carry the row's running maximum and sums across the column tiles.
extern "C" nova_status nova_head_entropy(nova_ctx* ctx, const void* x, const void* w_head, const void* b_head,
                                         int S, int N, int C, int V, float* ent, float* mean, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (S < 0 || N < 0 || C < 1 || V < 1) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_head_entropy: bad sizes");
    const long rows = (long)S * N;
    if (rows == 0) return NOVA_OK;
    if (rows > 0x7fffffffL) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_head_entropy: too many rows");
    if (!x || !w_head || !ent) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_head_entropy: null pointer");
    if (C % 64 || V % 32) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_head_entropy: C must be a multiple of 64 and V of 32");
    if (!nova_aligned16(x) || !nova_aligned16(w_head) || !nova_aligned16(b_head))
        return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_head_entropy: tensors must be 16-byte aligned");
    NOVA_DEVICE_GUARD(ctx, "nova_head_entropy");
    cudaStream_t st = (cudaStream_t)stream;
    nova_gemm_args g;
    memset(&g, 0, sizeof(g));
    g.A = (const __nv_bfloat16*)x; g.W = (const __nv_bfloat16*)w_head; g.bias = (const __nv_bfloat16*)b_head;
    g.M = (int)rows; g.N = V; g.K = C;
    g.epilogue = NOVA_EPI_ENTROPY; g.cat = NOVA_K_ENTROPY; g.ent = ent;
    const nova_status rc = nova_launch_gemm(ctx, g, st);
    if (rc) return rc;
    if (mean) {
        nova_launch_scope scope(ctx, NOVA_K_ENTROPY_MEAN, st);
        entropy_mean<<<S, 1024, 0, st>>>(ent, N, mean);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

// Eq. 4 / Eq. 7: per-token softmax entropy over the codebook logits and its per-image mean.
//
// One warp owns one row. The row is pulled from HBM exactly once with 128-bit loads and
// held in registers; the warp takes the row maximum, then one pass of exp2 gives
//   s = sum e^{z-m},  u = sum (z-m) e^{z-m},  H = ln s - u / s.
// Rows too wide for the register file fall back to a two-read streaming kernel.
// The mean is a second tiny kernel that sums in a fixed tree order (deterministic).
#include "common.cuh"

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

// finishing step shared by both kernels: lane 0 writes the row result
__device__ __forceinline__ void finish_row(float m, float s, float u, float* ent, long row,
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
}

__device__ __forceinline__ float fmax_nan(float a, float b)   // NaN if either input is NaN
{
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

// Per-lane running state of the streaming softmax-entropy: m = largest logit seen, s = sum of
// e^{z-m}, u = sum of (z-m) e^{z-m} (u kept in the log2 domain; m2 = m * log2 e). Raising m to m'
// multiplies both sums by f = e^{m-m'} and shifts u by (m-m') s:  u' = f (u + (m-m') s),  s' = f s.
struct RowState {
    float m, m2, s, u;
    __device__ __forceinline__ void raise_to(float m_new)
    {
        if (m == -INFINITY) { s = 0.f; u = 0.f; }
        else {
            const float shift = (m - m_new) * kLog2e;
            const float f = fast_exp2(shift);
            u = (u + shift * s) * f;
            s *= f;
        }
        m = m_new;
        m2 = m_new * kLog2e;
    }
    // One multiply-add, one clamp, one ex2, one add, one multiply-add per logit. The clamp turns a
    // -inf (or NaN) exponent into a huge negative finite one whose ex2 is exactly 0, so that it
    // contributes 0 instead of -inf * 0; NaN logits are caught by the NaN-propagating maximum.
    __device__ __forceinline__ void add(float z)
    {
        const float d = fmaxf(fmaf(z, kLog2e, -m2), -16000.f);
        const float e = fast_exp2(d);
        s += e;
        u = fmaf(d, e, u);
    }
};

// VEC = number of 16-byte vectors each lane holds. BF16: 8 values per vector; F32: 4.
// All loads of the row are issued before the first use (VEC * 16 bytes in flight per lane); the
// values stay packed in registers and are consumed once, vector by vector, by the streaming
// update above, so the register footprint is the packed row plus a handful of scalars.
template <int VEC, bool BF16>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
entropy_rows_reg(const void* __restrict__ logits, long rows, int V, long row_stride,
                 float* __restrict__ ent, unsigned int* status)
{
    constexpr int PER = BF16 ? 8 : 4;
    const int lane = threadIdx.x & 31;
    const long row = (long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int n_vec = V / PER;           // full vectors in the row (V % PER handled below)
    const char* base = (const char*)logits + row * row_stride * (BF16 ? 2 : 4);
    const uint4* src = (const uint4*)base;

    uint4 reg[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const int v = i * 32 + lane;
        if (v < n_vec) reg[i] = ld_stream(src + v);
        else reg[i] = BF16 ? make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u)   // -inf
                           : make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
    }
    // ragged tail (V not a multiple of the vector width): lane t takes element n_vec*PER + t
    float tail = -INFINITY;
    {
        const int e = n_vec * PER + lane;
        if (e < V) {
            tail = BF16 ? __bfloat162float(((const __nv_bfloat16*)base)[e]) : ((const float*)base)[e];
        }
    }

    RowState st;
    st.m = -INFINITY; st.m2 = -INFINITY; st.s = 0.f; st.u = 0.f;
    bool saw_nan = false;
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const uint32_t w[4] = {reg[i].x, reg[i].y, reg[i].z, reg[i].w};
        float cm;
        if (BF16) {
            // packed maximum: two logits per instruction
            __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&w[0]);
            __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&w[1]);
            __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162*>(&w[2]);
            __nv_bfloat162 d = *reinterpret_cast<const __nv_bfloat162*>(&w[3]);
            const __nv_bfloat162 mx = __hmax2_nan(__hmax2_nan(a, b), __hmax2_nan(c, d));
            const uint32_t mw = *reinterpret_cast<const uint32_t*>(&mx);
            float lo, hi;
            unpack_bf16x2(mw, lo, hi);
            cm = fmax_nan(lo, hi);
        } else {
            cm = fmax_nan(fmax_nan(__uint_as_float(w[0]), __uint_as_float(w[1])),
                          fmax_nan(__uint_as_float(w[2]), __uint_as_float(w[3])));
        }
        saw_nan |= (cm != cm);
        if (cm > st.m) st.raise_to(cm);             // rare after the first few vectors
        if (st.m != -INFINITY) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (BF16) {
                    float lo, hi;
                    unpack_bf16x2(w[q], lo, hi);
                    st.add(lo);
                    st.add(hi);
                } else {
                    st.add(__uint_as_float(w[q]));
                }
            }
        }
    }
    saw_nan |= (tail != tail);
    if (tail > st.m) st.raise_to(tail);
    if (st.m != -INFINITY) st.add(tail);

    // merge the 32 lanes: common maximum, then rescaled sums
    const float m = warp_max(st.m);
    float s = 0.f, u = 0.f;
    if (st.m != -INFINITY) {
        const float shift = (st.m - m) * kLog2e;
        const float f = fast_exp2(shift);
        s = st.s * f;
        u = (st.u + shift * st.s) * f;
        if (shift == -INFINITY) { s = 0.f; u = 0.f; }   // m = +inf: flagged below through m
    }
    if (saw_nan) s = __int_as_float(0x7fc00000);
    s = warp_sum(s);
    u = warp_sum(u);
    if (lane == 0) finish_row(m, s, u, ent, row, status);
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
    auto at = [&](int e) -> float {
        return BF16 ? __bfloat162float(((const __nv_bfloat16*)base)[e]) : ((const float*)base)[e];
    };
    float m = -INFINITY;
    for (int e = lane; e < V; e += 32) m = fmaxf(m, at(e));
    m = warp_max(m);
    float s = 0.f, u = 0.f;
    for (int e = lane; e < V; e += 32) {
        const float d = (at(e) - m) * kLog2e;
        const float ex = fast_exp2(d);
        s += ex;
        u = fmaf(d == -INFINITY ? 0.f : d, ex, u);
    }
    s = warp_sum(s);
    u = warp_sum(u);
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

}  // namespace

extern "C" nova_status nova_scale_entropy(nova_ctx* ctx, const void* logits, nova_dtype dt,
                                          int S, int N, int V, int64_t row_stride,
                                          float* ent, float* mean, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (S < 0 || N < 0 || V < 1 || (dt != NOVA_BF16 && dt != NOVA_F32))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_scale_entropy: bad S, N, V or dtype");
    const long rows = (long)S * N;
    if (rows == 0) return NOVA_OK;
    if (!logits || !ent) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_scale_entropy: null pointer");
    const int per = (dt == NOVA_BF16) ? 8 : 4;
    if (row_stride < V || (row_stride % per) != 0 || !nova_aligned16(logits))
        return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "nova_scale_entropy: logits rows must start on 16-byte boundaries");
    cudaStream_t st = (cudaStream_t)stream;
    {
        nova_launch_scope scope(ctx, NOVA_K_ENTROPY, st);
        if (dt == NOVA_BF16) launch_rows<true>(logits, rows, V, row_stride, ent, ctx->dev_status, st);
        else launch_rows<false>(logits, rows, V, row_stride, ent, ctx->dev_status, st);
    }
    if (mean) {
        nova_launch_scope scope(ctx, NOVA_K_ENTROPY_MEAN, st);
        entropy_mean<<<S, 1024, 0, st>>>(ent, N, mean);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

// Keep the k highest-entropy tokens of every segment (ties -> lower index) and build the
// gather/scatter index lists.
//
// One CTA per segment. The segment's keys (<= 16384 floats = 64 KiB) live in shared memory
// as order-preserving unsigned integers. A most-significant-digit radix select (4 passes of
// 8 bits, shared-memory histograms) finds the k-th largest key T and how many keys equal to
// T must still be taken; a final ordered pass (warp ballots + one block scan of the 32 warp
// totals) writes kept and pruned indices in ascending order.
#include "common.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxSegPerLaunch = 256;

struct SegParams {
    int32_t k[kMaxSegPerLaunch];
};

__device__ __forceinline__ uint32_t order_key(float f)
{
    uint32_t u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0;                       // -0 and +0 are the same key
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u); // larger float <=> larger key
}

// group == 0: the launch's segments form one list (cu_keep [S+1], kept and pruned lists concatenated
// over all segments). group > 0: every `group` consecutive segments (the images of one layer) form a
// list of their own: cumulative counts restart, group g writes cu_keep[g*(group+1) ...] and its index
// lists start at g*group*N. A launch then holds whole groups.
__global__ void __launch_bounds__(kThreads)
select_topk_kernel(const float* __restrict__ ent, int N, int seg0, int cu0, SegParams sp,
                   const int32_t* __restrict__ k_dev, int32_t* __restrict__ keep_idx, int32_t* __restrict__ prune_idx,
                   int32_t* __restrict__ cu_keep, int32_t* __restrict__ pos, int group)
{
    extern __shared__ uint32_t keys[];          // N keys
    __shared__ uint32_t hist[256];
    __shared__ uint32_t sh_prefix, sh_need;
    __shared__ uint32_t warp_gt[kWarps], warp_eq[kWarps];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int seg_local = blockIdx.x;
    const int seg = seg0 + seg_local;
    const int grp = group > 0 ? seg / group : 0;
    const int seg_in = group > 0 ? seg - grp * group : seg;          // position within its list
    const int list_first = seg - seg_in;                             // first segment of the list
    __shared__ int sh_cu;
    int k, cu;
    if (k_dev) {
        // keep counts written by an earlier kernel: clamp to [0, N]; cu = sum over the list's segments before
        if (tid == 0) sh_cu = 0;
        __syncthreads();
        int part = 0;
        for (int s = list_first + tid; s < seg; s += kThreads) part += min(max(k_dev[s], 0), N);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        if (lane == 0 && part) atomicAdd(&sh_cu, part);
        __syncthreads();
        cu = sh_cu;
        k = min(max(k_dev[seg], 0), N);
    } else {
        k = sp.k[seg_local];
        cu = group > 0 ? 0 : cu0;
        for (int s = group > 0 ? seg_local - seg_in : 0; s < seg_local; ++s) cu += sp.k[s];
    }
    if (tid == 0) {
        int32_t* cu_out = cu_keep + (group > 0 ? (long)grp * (group + 1) : 0);
        cu_out[seg_in] = cu;
        // last segment of a list (or of this launch: the next launch overwrites with the same value)
        if (group > 0 ? seg_in == group - 1 : seg_local == (int)gridDim.x - 1) cu_out[seg_in + 1] = cu + k;
    }

    const float* e = ent + (long)seg * N;
    for (int i = tid; i < N; i += kThreads) keys[i] = order_key(e[i]);

    // ---- radix select: threshold key T = k-th largest, need = how many keys == T are kept
    uint32_t prefix = 0, mask = 0, need = (uint32_t)k;
    if (k > 0 && k < N) {
        for (int shift = 24; shift >= 0; shift -= 8) {
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            for (int i = tid; i < N; i += kThreads) {
                const uint32_t key = keys[i];
                if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
            }
            __syncthreads();
            if (warp == 0) {
                // lane l owns digits 8l..8l+7; suffix sums from the top digit down
                uint32_t c[8], tot = 0;
#pragma unroll
                for (int d = 0; d < 8; ++d) { c[d] = hist[lane * 8 + d]; tot += c[d]; }
                // above = number of keys with a digit in a higher lane
                uint32_t incl = tot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t v = __shfl_down_sync(0xffffffffu, incl, o);
                    if (lane + o < 32) incl += v;
                }
                uint32_t above = incl - tot;
                // the digit we look for is the highest d with count(>d) < need <= count(>=d)
                if (above < need && need <= above + tot) {
#pragma unroll
                    for (int d = 7; d >= 0; --d) {
                        if (above < need && need <= above + c[d]) {
                            sh_prefix = prefix | ((uint32_t)(lane * 8 + d) << shift);
                            sh_need = need - above;
                            above = 0xffffffffu;   // stop
                        } else if (above != 0xffffffffu) {
                            above += c[d];
                        }
                    }
                }
            }
            __syncthreads();
            prefix = sh_prefix;
            need = sh_need;
            mask |= 255u << shift;
        }
    } else {
        __syncthreads();
    }
    // k == 0: keep nothing (threshold above every key); k == N: keep everything
    const bool keep_all = (k >= N), keep_none = (k <= 0);
    const uint32_t T = prefix;

    // ---- ordered emit. Warp w owns the contiguous index range [w*span, (w+1)*span).
    const int span = ((N + kWarps - 1) / kWarps + 31) & ~31;
    const int lo = warp * span, hi = min(N, lo + span);
    uint32_t n_gt = 0, n_eq = 0;
    for (int i0 = lo; i0 < hi; i0 += 32) {
        const int i = i0 + lane;
        const uint32_t key = (i < hi) ? keys[i] : 0u;
        const bool gt = (i < hi) && (keep_all || (!keep_none && key > T));
        const bool eq = (i < hi) && !keep_all && !keep_none && key == T;
        n_gt += __popc(__ballot_sync(0xffffffffu, gt));
        n_eq += __popc(__ballot_sync(0xffffffffu, eq));
    }
    if (lane == 0) { warp_gt[warp] = n_gt; warp_eq[warp] = n_eq; }
    __syncthreads();
    uint32_t gt_before = 0, eq_before = 0;
    for (int w2 = 0; w2 < warp; ++w2) { gt_before += warp_gt[w2]; eq_before += warp_eq[w2]; }

    const long list_base = (long)list_first * N;         // 0 unless grouped
    int32_t* keep_out = keep_idx + list_base + cu;
    int32_t* prune_out = prune_idx + list_base + ((long)seg_in * N - cu);
    int32_t* pos_out = pos ? pos + (long)seg * N : nullptr;
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int i0 = lo; i0 < hi; i0 += 32) {
        const int i = i0 + lane;
        const uint32_t key = (i < hi) ? keys[i] : 0u;
        const bool gt = (i < hi) && (keep_all || (!keep_none && key > T));
        const bool eq = (i < hi) && !keep_all && !keep_none && key == T;
        const uint32_t bg = __ballot_sync(0xffffffffu, gt);
        const uint32_t be = __ballot_sync(0xffffffffu, eq);
        const uint32_t my_gt = gt_before + __popc(bg & lt_mask);
        const uint32_t my_eq = eq_before + __popc(be & lt_mask);
        if (i < hi) {
            const bool kept = gt || (eq && my_eq < need);
            const uint32_t kept_before = my_gt + min(my_eq, need);
            if (kept) {
                keep_out[kept_before] = i;
                if (pos_out) pos_out[i] = (int32_t)kept_before;
            } else {
                prune_out[(uint32_t)i - kept_before] = i;
                if (pos_out) pos_out[i] = -1;
            }
        }
        gt_before += __popc(bg);
        eq_before += __popc(be);
    }
}

}  // namespace

extern "C" nova_status nova_select_topk(nova_ctx* ctx, const float* ent, int S, int N,
                                        const int32_t* k, int32_t* keep_idx, int32_t* prune_idx,
                                        int32_t* cu_keep, int32_t* pos, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (S < 0 || N < 0) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk: negative size");
    if (N > 16384) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_select_topk: N > 16384");
    if (!cu_keep) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk: null cu_keep");
    NOVA_DEVICE_GUARD(ctx, "nova_select_topk");
    cudaStream_t st = (cudaStream_t)stream;
    if (S == 0 || N == 0) {
        NOVA_CUDA_CHECK(ctx, cudaMemsetAsync(cu_keep, 0, sizeof(int32_t) * (size_t)(S + 1), st));
        return NOVA_OK;
    }
    if (!ent || !k) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk: null pointer");
    long total_keep = 0;
    for (int s = 0; s < S; ++s) {
        if (k[s] < 0 || k[s] > N) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk: k outside [0, N]");
        total_keep += k[s];
    }
    if ((total_keep > 0 && !keep_idx) || (total_keep < (long)S * N && !prune_idx))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk: null index output");

    if (!ctx->attr_select) {   // opt in to 64 KiB of dynamic shared memory once per context
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 16384 * 4));
        ctx->attr_select = true;
    }
    int cu = 0;
    for (int s0 = 0; s0 < S; s0 += kMaxSegPerLaunch) {
        const int n = (S - s0 < kMaxSegPerLaunch) ? (S - s0) : kMaxSegPerLaunch;
        SegParams sp;
        memset(&sp, 0, sizeof(sp));
        for (int s = 0; s < n; ++s) sp.k[s] = k[s0 + s];
        {
            nova_launch_scope scope(ctx, NOVA_K_SELECT, st);
            select_topk_kernel<<<n, kThreads, (size_t)N * 4, st>>>(ent, N, s0, cu, sp, nullptr, keep_idx, prune_idx, cu_keep, pos, 0);
        }
        for (int s = 0; s < n; ++s) cu += k[s0 + s];
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

// The same selection with the keep counts in device memory (written by nova_keep_ratios_device):
// no host value depends on them, so the call needs no synchronisation and can be captured.
extern "C" nova_status nova_select_topk_device(nova_ctx* ctx, const float* ent, int S, int N,
                                               const int32_t* k_dev, int32_t* keep_idx, int32_t* prune_idx,
                                               int32_t* cu_keep, int32_t* pos, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (S < 0 || N < 0) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk_device: negative size");
    if (N > 16384) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_select_topk_device: N > 16384");
    if (S > 65535) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_select_topk_device: S > 65535");
    if (!cu_keep) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk_device: null cu_keep");
    NOVA_DEVICE_GUARD(ctx, "nova_select_topk_device");
    cudaStream_t st = (cudaStream_t)stream;
    if (S == 0 || N == 0) {
        NOVA_CUDA_CHECK(ctx, cudaMemsetAsync(cu_keep, 0, sizeof(int32_t) * (size_t)(S + 1), st));
        return NOVA_OK;
    }
    if (!ent || !k_dev || !keep_idx || !prune_idx)
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk_device: null pointer");
    if (!ctx->attr_select) {
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 16384 * 4));
        ctx->attr_select = true;
    }
    SegParams sp;
    memset(&sp, 0, sizeof(sp));
    {
        nova_launch_scope scope(ctx, NOVA_K_SELECT, st);
        select_topk_kernel<<<S, kThreads, (size_t)N * 4, st>>>(ent, N, 0, 0, sp, k_dev, keep_idx, prune_idx, cu_keep, pos, 0);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

// Selection for all layers of a scale at once: G lists (layers) of S segments (images) each.
static nova_status select_grouped(nova_ctx* ctx, const float* ent, int G, int S, int N, const int32_t* k_host,
                                  const int32_t* k_dev, int32_t* keep_idx, int32_t* prune_idx, int32_t* cu_keep,
                                  int32_t* pos, void* stream, const char* who)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (G < 0 || S < 0 || N < 0) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk_grouped: negative size");
    if (N > 16384) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_select_topk_grouped: N > 16384");
    if (S > kMaxSegPerLaunch) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_select_topk_grouped: more than 256 segments per list");
    if ((long)G * S > 0x7fffffffL / (N > 0 ? N : 1)) return nova_fail(ctx, NOVA_ERR_SHAPE, "nova_select_topk_grouped: too many tokens");
    if (G == 0) return NOVA_OK;
    if (!cu_keep) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk_grouped: null cu_keep");
    NOVA_DEVICE_GUARD(ctx, who);
    cudaStream_t st = (cudaStream_t)stream;
    if (S == 0 || N == 0) {
        NOVA_CUDA_CHECK(ctx, cudaMemsetAsync(cu_keep, 0, sizeof(int32_t) * (size_t)G * (S + 1), st));
        return NOVA_OK;
    }
    if (!ent || (!k_host && !k_dev) || !keep_idx || !prune_idx)
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk_grouped: null pointer");
    if (k_host)
        for (long i = 0; i < (long)G * S; ++i)
            if (k_host[i] < 0 || k_host[i] > N)
                return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk_grouped: k outside [0, N]");
    if (!ctx->attr_select) {
        NOVA_CUDA_CHECK(ctx, cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 16384 * 4));
        ctx->attr_select = true;
    }
    SegParams sp;
    memset(&sp, 0, sizeof(sp));
    if (k_dev) {
        nova_launch_scope scope(ctx, NOVA_K_SELECT, st);
        select_topk_kernel<<<G * S, kThreads, (size_t)N * 4, st>>>(ent, N, 0, 0, sp, k_dev, keep_idx, prune_idx, cu_keep, pos, S);
    } else {
        // the host's counts travel as kernel parameters, 256 per launch: whole lists per launch
        const int lists_per_launch = kMaxSegPerLaunch / S;
        for (int g0 = 0; g0 < G; g0 += lists_per_launch) {
            const int ng = (G - g0 < lists_per_launch) ? (G - g0) : lists_per_launch;
            for (int i = 0; i < ng * S; ++i) sp.k[i] = k_host[(long)g0 * S + i];
            nova_launch_scope scope(ctx, NOVA_K_SELECT, st);
            select_topk_kernel<<<ng * S, kThreads, (size_t)N * 4, st>>>(ent, N, g0 * S, 0, sp, nullptr, keep_idx, prune_idx,
                                                                      cu_keep, pos, S);
        }
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

extern "C" nova_status nova_select_topk_grouped(nova_ctx* ctx, const float* ent, int G, int S, int N, const int32_t* k,
                                                int32_t* keep_idx, int32_t* prune_idx, int32_t* cu_keep,
                                                int32_t* pos, void* stream)
{
    if (ctx && G > 0 && S > 0 && N > 0 && !k) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk_grouped: null k");
    return select_grouped(ctx, ent, G, S, N, k, nullptr, keep_idx, prune_idx, cu_keep, pos, stream, "nova_select_topk_grouped");
}

extern "C" nova_status nova_select_topk_grouped_device(nova_ctx* ctx, const float* ent, int G, int S, int N,
                                                       const int32_t* k_dev, int32_t* keep_idx, int32_t* prune_idx,
                                                       int32_t* cu_keep, int32_t* pos, void* stream)
{
    if (ctx && G > 0 && S > 0 && N > 0 && !k_dev) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_select_topk_grouped_device: null k");
    return select_grouped(ctx, ent, G, S, N, nullptr, k_dev, keep_idx, prune_idx, cu_keep, pos, stream,
                          "nova_select_topk_grouped_device");
}

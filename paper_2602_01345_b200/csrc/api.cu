// Context management and the host-side schedule arithmetic (Eq. 8-13).
#include "tc_common.cuh"

#include <math.h>
#include <stdlib.h>
#include <new>

extern "C" {

const char* nova_status_string(nova_status s)
{
    switch (s) {
        case NOVA_OK: return "ok";
        case NOVA_ERR_INVALID_ARG: return "invalid argument";
        case NOVA_ERR_SHAPE: return "unsupported shape";
        case NOVA_ERR_ALIGNMENT: return "misaligned pointer or stride";
        case NOVA_ERR_WORKSPACE: return "workspace missing or too small";
        case NOVA_ERR_NONFINITE: return "non-finite logit";
        case NOVA_ERR_TIMEOUT: return "device-side wait expired";
        case NOVA_ERR_CUDA: return "CUDA error";
    }
    return "unknown status";
}

nova_status nova_create(nova_ctx** out, int device)
{
    if (!out) return NOVA_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess || device < 0 || device >= count) return NOVA_ERR_CUDA;
    nova_ctx* ctx = new (std::nothrow) nova_ctx();
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    ctx->device = device;
    ctx->dev_status = nullptr;
    ctx->workspace = nullptr;
    ctx->workspace_bytes = 0;
    ctx->encode_tiled = nullptr;
    ctx->num_sms = 0;
    ctx->attr_select = ctx->attr_gemm = ctx->attr_attn = false;
    ctx->err[0] = 0;
    ctx->launches = 0;
    ctx->profiling = false;
    ctx->prof_mask = ~0ull;
    ctx->events_used = 0;
    ctx->wait_limit_ns = 0;
    const char* dbg = getenv("NOVA_DEBUG");
    ctx->debug = dbg && dbg[0] && strcmp(dbg, "0") != 0;
    ctx->debug_failed = false;
    // the allocation is made with `device` current; the caller's current device is put back
    int prev = -1;
    const bool have_prev = (cudaGetDevice(&prev) == cudaSuccess);
    auto restore_device = [&]() { if (have_prev && prev != device) cudaSetDevice(prev); };
    if (cudaSetDevice(device) != cudaSuccess ||
        cudaMalloc(&ctx->dev_status, NOVA_STATUS_BYTES) != cudaSuccess ||
        cudaMemset(ctx->dev_status, 0, NOVA_STATUS_BYTES) != cudaSuccess) {
        delete ctx;
        restore_device();
        return NOVA_ERR_CUDA;
    }
    cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, device);
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaFree(ctx->dev_status);
        delete ctx;
        restore_device();
        return NOVA_ERR_CUDA;
    }
    ctx->encode_tiled = fn;
    restore_device();
    *out = ctx;
    return NOVA_OK;
}

void nova_destroy(nova_ctx* ctx)
{
    if (!ctx) return;
    int prev = -1;
    const bool have_prev = (cudaGetDevice(&prev) == cudaSuccess);
    cudaSetDevice(ctx->device);
    for (cudaEvent_t e : ctx->event_pool) cudaEventDestroy(e);
    cudaFree(ctx->dev_status);
    if (have_prev && prev != ctx->device) cudaSetDevice(prev);
    delete ctx;
}

unsigned long long nova_launch_count(const nova_ctx* ctx) { return ctx ? ctx->launches : 0; }

int nova_profile_categories(void) { return NOVA_K_COUNT; }

const char* nova_profile_category_name(int cat)
{
    static const char* names[NOVA_K_COUNT] = {
        "entropy_rows", "entropy_mean", "select_topk", "layernorm", "gemm_qkv",
        "attention", "gemm_proj", "gemm_fc1", "gemm_fc2", "restore", "keep_ratios", "selection_score"};
    return (cat >= 0 && cat < NOVA_K_COUNT) ? names[cat] : "?";
}

nova_status nova_profile_select(nova_ctx* ctx, unsigned long long category_mask)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    ctx->prof_mask = category_mask;
    return NOVA_OK;
}

nova_status nova_profile_begin(nova_ctx* ctx)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    ctx->prof_recs.clear();
    ctx->events_used = 0;
    ctx->profiling = true;
    return NOVA_OK;
}

nova_status nova_profile_end(nova_ctx* ctx, double* ms, long long* launches, int n)
{
    if (!ctx || !ms || !launches || n < NOVA_K_COUNT) return NOVA_ERR_INVALID_ARG;
    ctx->profiling = false;
    for (int i = 0; i < n; ++i) { ms[i] = 0.0; launches[i] = 0; }
    for (const nova_prof_rec& r : ctx->prof_recs) {
        NOVA_CUDA_CHECK(ctx, cudaEventSynchronize(r.stop));
        float t = 0.f;
        NOVA_CUDA_CHECK(ctx, cudaEventElapsedTime(&t, r.start, r.stop));
        ms[r.cat] += (double)t;
        launches[r.cat] += 1;
    }
    ctx->prof_recs.clear();
    ctx->events_used = 0;
    return NOVA_OK;
}

const char* nova_last_error(const nova_ctx* ctx) { return ctx ? ctx->err : "null context"; }

nova_status nova_device_status(nova_ctx* ctx, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    NOVA_DEVICE_GUARD(ctx, "nova_device_status");
    cudaStream_t st = (cudaStream_t)stream;
    unsigned int word = 0;
    NOVA_CUDA_CHECK(ctx, cudaMemcpyAsync(&word, ctx->dev_status, sizeof(word), cudaMemcpyDeviceToHost, st));
    NOVA_CUDA_CHECK(ctx, cudaStreamSynchronize(st));
    // an aborted kernel may leave the entropy accumulators or attention tickets half way: clear everything
    if (word) {
        NOVA_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->dev_status, 0, NOVA_STATUS_BYTES, st));
        if (ctx->wait_limit_ns)     // the wait limit lives in the same block: put it back
            NOVA_CUDA_CHECK(ctx, cudaMemcpyAsync(ctx->dev_status + NOVA_WAIT_LIMIT_WORD, &ctx->wait_limit_ns,
                                                 sizeof(ctx->wait_limit_ns), cudaMemcpyHostToDevice, st));
        NOVA_CUDA_CHECK(ctx, cudaStreamSynchronize(st));
    }
    if (ctx->debug_failed) {    // message already in err: a launch failed under debug mode's per-launch synchronisation
        ctx->debug_failed = false;
        return NOVA_ERR_CUDA;
    }
    if (word & NOVA_DEV_TIMEOUT) return nova_fail(ctx, NOVA_ERR_TIMEOUT, "a device-side wait expired");
    if (word & NOVA_DEV_BAD_INDEX) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "an index list failed the debug mode's validation");
    if (word & NOVA_DEV_SHAPE) return nova_fail(ctx, NOVA_ERR_SHAPE, "K/V cache overflow on the device");
    if (word & NOVA_DEV_NONFINITE) return nova_fail(ctx, NOVA_ERR_NONFINITE, "non-finite logit");
    return NOVA_OK;
}

nova_status nova_set_wait_limit_ns(nova_ctx* ctx, unsigned long long ns)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    NOVA_DEVICE_GUARD(ctx, "nova_set_wait_limit_ns");
    ctx->wait_limit_ns = ns;
    // ordered after everything enqueued so far on any stream: a synchronous copy
    NOVA_CUDA_CHECK(ctx, cudaDeviceSynchronize());
    NOVA_CUDA_CHECK(ctx, cudaMemcpy(ctx->dev_status + NOVA_WAIT_LIMIT_WORD, &ctx->wait_limit_ns, sizeof(ns), cudaMemcpyHostToDevice));
    return NOVA_OK;
}

nova_status nova_set_debug(nova_ctx* ctx, int on)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    ctx->debug = on != 0;
    return NOVA_OK;
}

}  // extern "C"

// Debug mode: one block per segment validates that segment's slice of the lists. A block touches a
// list only after its own two prefix-sum entries have passed, so that no read leaves the lists.
__global__ void check_lists_kernel(const int32_t* __restrict__ keep_idx, const int32_t* __restrict__ prune_idx,
                                   const int32_t* __restrict__ cu_keep, int N, long m_bound, bool m_exact,
                                   unsigned int* status)
{
    const int s = blockIdx.x;
    const long c0 = cu_keep[s], c1 = cu_keep[s + 1];
    bool bad = (s == 0 && c0 != 0) || c0 < 0 || c0 > (long)s * N || c1 < c0 || c1 - c0 > N || c1 > m_bound ||
               (m_exact && s == (int)gridDim.x - 1 && c1 != m_bound);
    if (!bad) {
        if (keep_idx) {
            for (long i = c0 + threadIdx.x; i < c1; i += blockDim.x) {
                const int v = keep_idx[i];
                if (v < 0 || v >= N || (i > c0 && keep_idx[i - 1] >= v)) bad = true;
            }
        }
        if (prune_idx) {
            const long p0 = (long)s * N - c0, p1 = p0 + N - (c1 - c0);
            for (long i = p0 + threadIdx.x; i < p1; i += blockDim.x) {
                const int v = prune_idx[i];
                if (v < 0 || v >= N || (i > p0 && prune_idx[i - 1] >= v)) bad = true;
            }
        }
    }
    if (bad) atomicOr(status, NOVA_DEV_BAD_INDEX);
}

nova_status nova_debug_check_lists(nova_ctx* ctx, const char* who, const int32_t* keep_idx,
                                   const int32_t* prune_idx, const int32_t* cu_keep,
                                   int B, int N, long m_bound, bool m_exact, cudaStream_t st)
{
    if (!ctx->debug || B <= 0 || !cu_keep) return NOVA_OK;
    check_lists_kernel<<<B, 256, 0, st>>>(keep_idx, prune_idx, cu_keep, N, m_bound, m_exact, ctx->dev_status);
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    unsigned int word = 0;
    NOVA_CUDA_CHECK(ctx, cudaMemcpyAsync(&word, ctx->dev_status, sizeof(word), cudaMemcpyDeviceToHost, st));
    NOVA_CUDA_CHECK(ctx, cudaStreamSynchronize(st));
    if (word & NOVA_DEV_BAD_INDEX) {
        word &= ~NOVA_DEV_BAD_INDEX;
        NOVA_CUDA_CHECK(ctx, cudaMemcpyAsync(ctx->dev_status, &word, sizeof(word), cudaMemcpyHostToDevice, st));
        NOVA_CUDA_CHECK(ctx, cudaStreamSynchronize(st));
        snprintf(ctx->err, sizeof(ctx->err), "%s: keep_idx / prune_idx / cu_keep failed validation (debug mode): nothing launched", who);
        return NOVA_ERR_INVALID_ARG;
    }
    return NOVA_OK;
}

extern "C" {

// One CTA whose consumer warp waits on a barrier that no producer ever arrives on: the wait runs
// into the context's limit, records the time-out and the kernel returns normally.
__global__ void wait_probe_kernel(unsigned int* status)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;
    if (threadIdx.x == 0) {
        abort_flag_s = 0;
        tc::mbar_init(&bar, 1);
        tc::fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x < 32) tc::mbar_wait_warp(&bar, 0, abort_flag, status);
    __syncthreads();
}

nova_status nova_debug_wait_probe(nova_ctx* ctx, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    NOVA_DEVICE_GUARD(ctx, "nova_debug_wait_probe");
    wait_probe_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(ctx->dev_status);
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

nova_status nova_set_workspace(nova_ctx* ctx, void* dev_ptr, size_t bytes)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (dev_ptr && (((uintptr_t)dev_ptr) & 255u)) return nova_fail(ctx, NOVA_ERR_ALIGNMENT, "workspace must be 256-byte aligned");
    ctx->workspace = dev_ptr;
    ctx->workspace_bytes = dev_ptr ? bytes : 0;
    return NOVA_OK;
}

void nova_sched_params_default(nova_sched_params* p)
{
    if (!p) return;
    p->t_est = 5;
    p->alpha = 0.5;
    p->tau = 0.8;
    p->lambda = 0.1;
    p->k_min = 1;
    p->ratio_max = 1.0;
    p->force_act_scale = 0;
    p->force_keep_ratio = -1.0;
}

// Eq. 8-13 for one image. HS(u) is the mean entropy of scale u, HL(k) that of layer k; the
// histories are strided so that the host layout [B, t] and the device layout [t, B] share the code.
static __host__ __device__ void schedule_one(const nova_sched_params& p, int t, int j, int n_tokens,
                                             const float* hs_base, long hs_stride, const float* hl_base, long hl_stride,
                                             int32_t* t_star, int32_t* act_scale, double* ratio_scale,
                                             double* ratio_layer, int32_t* keep)
{
#define HS(u) ((double)hs_base[((u) - 1) * hs_stride])
#define HL(k) ((double)hl_base[((k) - 1) * hl_stride])
    // growth rates g[u] for u = 2..t (Eq. 8)
    double growth_now = 0.0;
    int found = 0;
    if (t > p.t_est) {
        // baseline: the growth rates up to t_est telescope, but are summed one by one so the
        // rounding matches a term-by-term evaluation of Eq. 9
        double base = 0.0;
        for (int u = 2; u <= p.t_est; ++u) base += HS(u) - HS(u - 1);
        base /= (double)(p.t_est - 1);
        const double threshold = p.alpha * base;
        for (int u = p.t_est + 1; u <= t && !found; ++u) {
            const double gu = HS(u) - HS(u - 1);
            const double gprev = HS(u - 1) - HS(u - 2);
            if ((gu + gprev) / 2.0 <= threshold) found = u;   // Eq. 10
        }
    }
    int act = found ? found + 1 : 0;
    if (p.force_act_scale > 0) {
        act = p.force_act_scale;
        found = act - 1;
    }
    *t_star = found;
    *act_scale = act;

    double rs = 0.0, rl = 0.0;
    if (act > 0 && t >= act) {
        if (p.force_keep_ratio >= 0.0) {
            rs = rl = 1.0 - p.force_keep_ratio;
        } else {
            if (t >= 2) growth_now = HS(t) - HS(t - 1);
            const double arg = ((double)t - (double)act) / p.tau;
            rs = 1.0 / (1.0 + exp(-arg)) - p.lambda * tanh(growth_now);   // Eq. 11
            rl = rs;
            if (j >= 2) {                                                // Eq. 12-13
                double mu = 0.0;
                for (int k = 1; k < j; ++k) mu += HL(k);
                mu /= (double)(j - 1);
                const double delta = (mu != 0.0) ? (HL(j) - mu) / mu : 0.0;
                rl = rs - delta * rs;
            }
        }
    }
    *ratio_scale = rs;
    *ratio_layer = rl;
    double r = rl < 0.0 ? 0.0 : rl;
    if (r > p.ratio_max) r = p.ratio_max;
    long kept = (long)n_tokens - (long)floor(r * (double)n_tokens);
    if (kept < p.k_min) kept = p.k_min;
    if (kept > n_tokens) kept = n_tokens;
    *keep = (int32_t)kept;
#undef HS
#undef HL
}

// One thread per image; the histories are device arrays [t, B] and [j, B].
__global__ void keep_ratios_kernel(const nova_sched_params p, int B, int t, int j, int n_tokens,
                                   const float* __restrict__ hs, const float* __restrict__ hl,
                                   int32_t* __restrict__ t_star, int32_t* __restrict__ act_scale,
                                   int32_t* __restrict__ keep)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int32_t ts, as, kp;
    double rs, rl;
    schedule_one(p, t, j, n_tokens, hs + b, B, hl ? hl + b : nullptr, B, &ts, &as, &rs, &rl, &kp);
    if (t_star) t_star[b] = ts;
    if (act_scale) act_scale[b] = as;
    keep[b] = kp;
}

// All L layers of a scale at once; thread (j, b) evaluates layer j + 1 of image b on the means of
// layers 1..j+1 (every layer's mean is known once the scale's entropy maps are taken).
__global__ void keep_ratios_layers_kernel(const nova_sched_params p, int B, int t, int L, int n_tokens,
                                          const float* __restrict__ hs, const float* __restrict__ hl,
                                          int32_t* __restrict__ t_star, int32_t* __restrict__ act_scale,
                                          int32_t* __restrict__ keep)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= L * B) return;
    const int j = i / B, b = i - j * B;
    int32_t ts, as, kp;
    double rs, rl;
    schedule_one(p, t, j + 1, n_tokens, hs + b, B, hl + b, B, &ts, &as, &rs, &rl, &kp);
    if (j == 0) {
        if (t_star) t_star[b] = ts;
        if (act_scale) act_scale[b] = as;
    }
    keep[i] = kp;
}

nova_status nova_keep_ratios_layers(const nova_sched_params* p, int B, int t, int L, int N_t,
                                    const float* hbar_scale, const float* hbar_layer,
                                    int32_t* t_star, int32_t* act_scale,
                                    double* ratio_scale, double* ratio_layer, int32_t* keep)
{
    if (!p || B < 0 || t < 1 || L < 1 || N_t < 1 || p->t_est < 2 || !(p->tau > 0.0)) return NOVA_ERR_INVALID_ARG;
    if (B == 0) return NOVA_OK;
    if (!hbar_scale || !hbar_layer || !t_star || !act_scale || !ratio_scale || !ratio_layer || !keep) return NOVA_ERR_INVALID_ARG;
    for (int j = 0; j < L; ++j)
        for (int b = 0; b < B; ++b)
            schedule_one(*p, t, j + 1, N_t, hbar_scale + (size_t)b * t, 1, hbar_layer + (size_t)b * L, 1,
                         t_star + b, act_scale + b, ratio_scale + b, ratio_layer + (size_t)j * B + b, keep + (size_t)j * B + b);
    return NOVA_OK;
}

nova_status nova_keep_ratios_layers_device(nova_ctx* ctx, const nova_sched_params* p, int B, int t, int L, int N_t,
                                           const float* hbar_scale, const float* hbar_layer,
                                           int32_t* t_star, int32_t* act_scale, int32_t* keep, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (!p || B < 0 || t < 1 || L < 1 || N_t < 1 || p->t_est < 2 || !(p->tau > 0.0))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_keep_ratios_layers_device: bad argument");
    if (B == 0) return NOVA_OK;
    if (!hbar_scale || !hbar_layer || !keep)
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_keep_ratios_layers_device: null pointer");
    NOVA_DEVICE_GUARD(ctx, "nova_keep_ratios_layers_device");
    cudaStream_t st = (cudaStream_t)stream;
    {
        nova_launch_scope scope(ctx, NOVA_K_KEEP_RATIOS, st);
        keep_ratios_layers_kernel<<<(L * B + 127) / 128, 128, 0, st>>>(*p, B, t, L, N_t, hbar_scale, hbar_layer, t_star,
                                                                     act_scale, keep);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

nova_status nova_keep_ratios(const nova_sched_params* p, int B, int t, int j, int N_t,
                             const float* hbar_scale, const float* hbar_layer,
                             int32_t* t_star, int32_t* act_scale,
                             double* ratio_scale, double* ratio_layer, int32_t* keep)
{
    if (!p || B < 0 || t < 1 || j < 1 || N_t < 1 || p->t_est < 2 || !(p->tau > 0.0)) return NOVA_ERR_INVALID_ARG;
    if (B == 0) return NOVA_OK;
    if (!hbar_scale || !t_star || !act_scale || !ratio_scale || !ratio_layer || !keep) return NOVA_ERR_INVALID_ARG;
    if (j >= 2 && !hbar_layer && p->force_keep_ratio < 0.0) return NOVA_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b)
        schedule_one(*p, t, j, N_t, hbar_scale + (size_t)b * t, 1,
                     hbar_layer ? hbar_layer + (size_t)b * j : nullptr, 1,
                     t_star + b, act_scale + b, ratio_scale + b, ratio_layer + b, keep + b);
    return NOVA_OK;
}

nova_status nova_keep_ratios_device(nova_ctx* ctx, const nova_sched_params* p, int B, int t, int j, int N_t,
                                    const float* hbar_scale, const float* hbar_layer,
                                    int32_t* t_star, int32_t* act_scale, int32_t* keep, void* stream)
{
    if (!ctx) return NOVA_ERR_INVALID_ARG;
    if (!p || B < 0 || t < 1 || j < 1 || N_t < 1 || p->t_est < 2 || !(p->tau > 0.0))
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_keep_ratios_device: bad argument");
    if (B == 0) return NOVA_OK;
    if (!hbar_scale || !keep) return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_keep_ratios_device: null pointer");
    if (j >= 2 && !hbar_layer && p->force_keep_ratio < 0.0)
        return nova_fail(ctx, NOVA_ERR_INVALID_ARG, "nova_keep_ratios_device: layer history missing");
    NOVA_DEVICE_GUARD(ctx, "nova_keep_ratios_device");
    cudaStream_t st = (cudaStream_t)stream;
    {
        nova_launch_scope scope(ctx, NOVA_K_KEEP_RATIOS, st);
        keep_ratios_kernel<<<(B + 127) / 128, 128, 0, st>>>(*p, B, t, j, N_t, hbar_scale, hbar_layer, t_star,
                                                           act_scale, keep);
    }
    NOVA_CUDA_CHECK(ctx, cudaGetLastError());
    return NOVA_OK;
}

}  // extern "C"

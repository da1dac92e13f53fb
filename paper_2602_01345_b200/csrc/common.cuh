// Shared host/device declarations of the NOVA CUDA library (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>
#include <vector>
#include <nvtx3/nvToolsExt.h>

#include "../../include/nova.h"

// Device status word: kernels OR these bits in; nova_device_status() maps them to a status.
#define NOVA_DEV_NONFINITE 1u
#define NOVA_DEV_TIMEOUT   2u
#define NOVA_DEV_SHAPE     4u
#define NOVA_DEV_BAD_INDEX 8u         // set by the debug mode's validation of keep / prune / cu_keep lists

// Layout of the context's one device allocation: NOVA_STATUS_WORDS 32-bit words (word 0 = status
// flags, a block of tickets for key-split attention items), then one 64-bit accumulator per segment
// for the entropy means (NOVA_MEAN_MAX_SEGMENTS of them). All of it is zero between launches.
#define NOVA_STATUS_WORDS 128
#define NOVA_WAIT_LIMIT_WORD 2        // words 2-3: limit of a device-side wait in ns (0 = the default of one second)
#define NOVA_ATTN_TICKET_WORD0 16     // words 16 .. 16 + NOVA_ATTN_TICKETS - 1: tickets of key-split attention items
#define NOVA_ATTN_TICKETS 96
#define NOVA_MEAN_MAX_CTAS 192        // the accumulator's arrival count has 8 bits
#define NOVA_MEAN_MAX_SEGMENTS 256
#define NOVA_STATUS_BYTES (NOVA_STATUS_WORDS * 4 + NOVA_MEAN_MAX_SEGMENTS * 8)

// Kernel categories for the launch counter and the optional per-kernel event timing.
enum nova_kernel_cat {
    NOVA_K_ENTROPY = 0, NOVA_K_ENTROPY_MEAN, NOVA_K_SELECT, NOVA_K_LAYERNORM,
    NOVA_K_GEMM_QKV, NOVA_K_ATTENTION, NOVA_K_GEMM_PROJ, NOVA_K_GEMM_FC1, NOVA_K_GEMM_FC2,
    NOVA_K_RESTORE, NOVA_K_KEEP_RATIOS, NOVA_K_SCORE, NOVA_K_COUNT
};

struct nova_prof_rec {
    int cat;
    cudaEvent_t start, stop;
};

struct nova_ctx {
    int device;
    unsigned int* dev_status;   // one word of device memory
    void* workspace;            // caller-owned device scratch
    size_t workspace_bytes;
    void* encode_tiled;         // cuTensorMapEncodeTiled, resolved through the runtime
    int num_sms;
    bool attr_select, attr_gemm, attr_attn;   // dynamic shared memory opt-in done on this device
    unsigned long long wait_limit_ns;   // mirrored in the status block (0 = default)
    bool debug;                 // debug mode: index lists validated before use, every launch synchronised
    bool debug_failed;          // a launch failed in debug mode (message in err); reported by nova_device_status
    char err[256];
    // measurement: launches since creation, and event pairs around each launch while profiling
    unsigned long long launches;
    bool profiling;
    unsigned long long prof_mask;             // categories that get event brackets while profiling (bit c = category c)
    std::vector<nova_prof_rec> prof_recs;     // records of the current profiling window
    std::vector<cudaEvent_t> event_pool;      // events created so far (reused across windows)
    size_t events_used;
};

// Brackets one kernel launch: counts it and, while profiling, records events around it on the
// launching stream.
struct nova_launch_scope {
    nova_ctx* ctx;
    cudaStream_t st;
    cudaEvent_t stop;
    nova_launch_scope(nova_ctx* c, int cat, cudaStream_t s) : ctx(c), st(s), stop(nullptr)
    {
        ctx->launches++;
        if (!ctx->profiling || !((ctx->prof_mask >> cat) & 1ull)) return;
        while (ctx->event_pool.size() < ctx->events_used + 2) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) return;
            ctx->event_pool.push_back(e);
        }
        nova_prof_rec r;
        r.cat = cat;
        r.start = ctx->event_pool[ctx->events_used++];
        r.stop = ctx->event_pool[ctx->events_used++];
        cudaEventRecord(r.start, st);
        ctx->prof_recs.push_back(r);
        stop = r.stop;
    }
    ~nova_launch_scope()
    {
        if (stop) cudaEventRecord(stop, st);
        if (ctx->debug && !ctx->debug_failed) {
            // debug mode: an asynchronous failure is pinned to the launch that caused it
            const cudaError_t e = cudaStreamSynchronize(st);
            if (e != cudaSuccess) {
                snprintf(ctx->err, sizeof(ctx->err), "launch %llu failed: %s", ctx->launches, cudaGetErrorString(e));
                ctx->debug_failed = true;
            }
        }
    }
};

// One NVTX range per C-ABI call (a no-op unless a tool that listens to NVTX is attached).
struct nova_api_range {
    explicit nova_api_range(const char* name) { nvtxRangePushA(name); }
    ~nova_api_range() { nvtxRangePop(); }
    nova_api_range(const nova_api_range&) = delete;
    nova_api_range& operator=(const nova_api_range&) = delete;
};

static inline nova_status nova_fail(nova_ctx* ctx, nova_status s, const char* msg)
{
    if (ctx) {
        strncpy(ctx->err, msg, sizeof(ctx->err) - 1);
        ctx->err[sizeof(ctx->err) - 1] = 0;
    }
    return s;
}

static inline nova_status nova_cuda_fail(nova_ctx* ctx, cudaError_t e, const char* where)
{
    if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s: %s", where, cudaGetErrorString(e));
    return NOVA_ERR_CUDA;
}

#define NOVA_CUDA_CHECK(ctx, expr)                                            \
    do {                                                                      \
        cudaError_t e__ = (expr);                                             \
        if (e__ != cudaSuccess) return nova_cuda_fail((ctx), e__, #expr);     \
    } while (0)

static inline bool nova_aligned16(const void* p) { return (((uintptr_t)p) & 15u) == 0; }

// Every launching entry point runs on the caller's current device with pointers (status word,
// workspace) that live on the context's device: refuse the call when the two differ instead of
// letting a kernel dereference another GPU's memory.
static inline nova_status nova_check_device(nova_ctx* ctx, const char* who)
{
    int cur = -1;
    const cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) return nova_cuda_fail(ctx, e, "cudaGetDevice");
    if (cur != ctx->device) {
        snprintf(ctx->err, sizeof(ctx->err), "%s: the context belongs to device %d but device %d is current",
                 who, ctx->device, cur);
        return NOVA_ERR_INVALID_ARG;
    }
    return NOVA_OK;
}
// Also opens the call's NVTX range, which lasts until the calling function returns.
#define NOVA_DEVICE_GUARD(ctx, who)                                           \
    nova_api_range nova_api_range__(who);                                     \
    do {                                                                      \
        const nova_status g__ = nova_check_device((ctx), (who));              \
        if (g__ != NOVA_OK) return g__;                                       \
    } while (0)

// Debug mode only (returns NOVA_OK at once otherwise): checks on the device, before any kernel uses
// them, that cu_keep is a valid prefix sum (cu_keep[0] = 0, 0 <= k_s <= N, total <= m_bound, or
// == m_bound when m_exact) and that every keep / prune entry is an in-segment index in [0, N),
// ascending within its segment. Synchronises the stream. keep_idx or prune_idx may be null (that
// list is then not looked at).
nova_status nova_debug_check_lists(nova_ctx* ctx, const char* who, const int32_t* keep_idx,
                                   const int32_t* prune_idx, const int32_t* cu_keep,
                                   int B, int N, long m_bound, bool m_exact, cudaStream_t st);

// Kernel launchers implemented in the other translation units.

enum nova_epilogue {
    NOVA_EPI_QKV = 0,       // +bias; columns [0,C) -> q, [C,2C) -> k cache rows, [2C,3C) -> v cache rows
    NOVA_EPI_BIAS_RES = 1,  // +bias + residual[res_row[r]] -> out
    NOVA_EPI_BIAS_GELU = 2, // GELU_tanh(+bias) -> out
    NOVA_EPI_ENTROPY = 3    // +bias (optional); nothing stored but ent[r] = entropy of softmax(row r) over all N columns
};

struct nova_gemm_args {
    const __nv_bfloat16* A;     // [M, K] row-major
    const __nv_bfloat16* W;     // [N, K] row-major
    const __nv_bfloat16* bias;  // [N]
    int M, N, K;
    const int32_t* m_dev;       // NULL, or device: the true row count (<= M, which then sizes the grid and maps)
    int epilogue;
    int cat;                    // nova_kernel_cat of this launch
    __nv_bfloat16* out;         // [M, N] (QKV: q buffer [M, C])
    // residual epilogue
    const __nv_bfloat16* res;   // residual rows of width N
    const int32_t* res_row;     // row map into res, or NULL for identity
    const __nv_bfloat16* gate;  // NULL, or [images, N]: out = res + gate[img_row[r]] * (acc + bias)
    const int32_t* img_row;     // [M] image of each row (needed with gate)
    // scattered output (residual epilogue only): row r goes to row out_row[r] of `out`, and, with
    // diff_out, diff_out[out_row[r]] = out value - diff_in[out_row[r]] (Eq. 15 on the kept rows)
    const int32_t* out_row;
    const __nv_bfloat16* diff_in;
    __nv_bfloat16* diff_out;
    // QKV epilogue
    int C;
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    const int32_t* kv_row;      // [M] destination cache row (b*Lmax + kv_len[b] + m), -1 = skip
    float* ent;                 // entropy epilogue: [M] fp32
    // optional tail of the launch: kv_len[b] += cu_keep[b+1] - cu_keep[b] where it fits in Lmax
    const int32_t* adv_cu_keep;
    int32_t* adv_kv_len;
    int adv_B, adv_Lmax;
};

nova_status nova_launch_gemm(nova_ctx* ctx, const nova_gemm_args& a, cudaStream_t st);

struct nova_attn_args {
    const __nv_bfloat16* q;        // [M, C]
    const __nv_bfloat16* k_cache;  // [B, Lmax, C] already holding the new rows
    const __nv_bfloat16* v_cache;
    const int32_t* cu_keep;        // [B+1]
    const int32_t* kv_len;         // [B] length before this call's rows
    __nv_bfloat16* o;              // [M, C]
    int B, C, n_heads, Lmax, M;
    void* scratch;                 // device memory free during the launch (or NULL) for a key-split last wave
    size_t scratch_bytes;
    bool cache_only;               // cross-attention: the keys are the kv_len[b] cache rows alone (no rows of this call)
};

nova_status nova_launch_attention(nova_ctx* ctx, const nova_attn_args& a, cudaStream_t st);

// Eq. 16 for the pruned rows only (restore.cu); the kept rows were written by the block's last epilogue.
nova_status nova_restore_pruned_rows(nova_ctx* ctx, const void* x_in, const int32_t* prune_idx,
                                     const int32_t* cu_keep, const void* cache_prev,
                                     int hp, int wp, int h, int w, int C, int B, int M, bool m_on_device,
                                     void* x_out, void* cache_out, void* stream);

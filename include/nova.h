/*
 * nova.h - C ABI of the NOVA pruned-scale step for one NVIDIA B200 (sm_100a).
 *
 * The library runs the work that NOVA (training-free acceleration of next-scale
 * visual autoregressive generation) adds to, and removes from, one transformer layer
 * at an accelerated scale:
 *
 *   nova_scale_entropy      Eq. 4, Eq. 7   per-token entropy and per-image mean
 *   nova_head_entropy       Eq. 4, Eq. 7   the same from hidden states and the codebook head
 *   nova_keep_ratios        Eq. 8-13       inflection trigger, scale/layer ratios, keep counts
 *   nova_select_topk        text after Eq. 3 / Eq. 13: keep the highest-entropy tokens
 *   nova_pruned_block_forward   Eq. 14     the layer on the kept tokens only
 *   nova_restore_from_cache     Eq. 15-16  fill pruned rows from the residual cache
 *   nova_*_device               the same steps with the keep counts left on the device
 *
 * General rules
 *  - Plain C ABI. No call throws, aborts or traps the GPU. Every call returns a
 *    nova_status; nova_last_error() gives a text for the last failure on a context.
 *  - "device" pointers are CUDA device pointers owned by the caller; "host" pointers
 *    are ordinary host memory owned by the caller. The library never frees or keeps
 *    a caller pointer beyond the call, except the workspace given to
 *    nova_set_workspace(), which it uses until replaced or the context is destroyed.
 *  - All device work is enqueued on the `stream` argument (a cudaStream_t passed as
 *    void*; NULL is the legacy default stream) and is asynchronous with respect to
 *    the host. Calls on one context must not overlap on the GPU: they share the
 *    workspace and the device status word.
 *  - bf16 tensors are row-major with the last dimension contiguous; device pointers to
 *    bf16/f32 tensors must be 16-byte aligned. Index tensors are int32.
 *  - Scales t and layers j are 1-based as in the paper.
 *  - A context belongs to one CUDA device, which must be the caller's current device at every
 *    call that enqueues work (else NOVA_ERR_INVALID_ARG; nothing is launched). nova_create and
 *    nova_destroy leave the caller's current device as they found it.
 *  - Device-side waits are bounded. If one expires the kernel records
 *    NOVA_ERR_TIMEOUT in the context's device status word and returns; non-finite
 *    logits record NOVA_ERR_NONFINITE. nova_device_status() reads that word.
 */
#ifndef NOVA_H
#define NOVA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct nova_ctx nova_ctx;

typedef enum nova_status {
    NOVA_OK = 0,
    NOVA_ERR_INVALID_ARG = 1,  /* null pointer, negative count, bad enum            */
    NOVA_ERR_SHAPE = 2,        /* size outside what the kernels support             */
    NOVA_ERR_ALIGNMENT = 3,    /* pointer or stride not 16-byte aligned             */
    NOVA_ERR_WORKSPACE = 4,    /* workspace missing or too small                    */
    NOVA_ERR_NONFINITE = 5,    /* +inf or NaN logit seen (device status)            */
    NOVA_ERR_TIMEOUT = 6,      /* a bounded device-side wait expired (device status)*/
    NOVA_ERR_CUDA = 7          /* a CUDA runtime/driver call failed                 */
} nova_status;

typedef enum nova_dtype { NOVA_BF16 = 0, NOVA_F32 = 1 } nova_dtype;

/* ---- context ------------------------------------------------------------------ */

/* Creates a context bound to CUDA device `device`. Allocates about 3 KB of device memory for
 * the status word, tickets and the accumulators of the entropy means (the only allocation the
 * library ever makes). */
nova_status nova_create(nova_ctx** out, int device);
void        nova_destroy(nova_ctx* ctx);
const char* nova_last_error(const nova_ctx* ctx);
const char* nova_status_string(nova_status s);

/* Synchronises `stream`, returns the device status word (NOVA_OK, NOVA_ERR_TIMEOUT,
 * NOVA_ERR_SHAPE for a K/V cache that would overflow, or NOVA_ERR_NONFINITE, in that order of
 * precedence; in debug mode also NOVA_ERR_CUDA for a launch that failed) and clears it. */
nova_status nova_device_status(nova_ctx* ctx, void* stream);

/* ---- bounded device-side waits (no counterpart in the paper) -------------------- */
/* Every wait inside a kernel (on a copy in flight, on another warp, on the tensor core) gives up
 * after a limit, records NOVA_ERR_TIMEOUT in the device status word and lets the kernel return, so
 * that a lost signal can never hang the GPU. nova_set_wait_limit_ns sets that limit for the
 * context's later launches (0 = the default, one second); it synchronises the device.
 * nova_debug_wait_probe launches a one-block diagnostic kernel whose only warp waits for a signal
 * that never comes: it must return after the limit with NOVA_ERR_TIMEOUT in the status word and
 * leave the context usable. It reads and writes no caller memory. */
nova_status nova_set_wait_limit_ns(nova_ctx* ctx, unsigned long long ns);
nova_status nova_debug_wait_probe(nova_ctx* ctx, void* stream);

/* ---- debug mode and tracing (no counterpart in the paper) ------------------------ */
/* Debug mode is off unless the environment variable NOVA_DEBUG is set (and not "0") when the
 * context is created; nova_set_debug switches it for the context's later calls. While it is on,
 *  - every call that reads index lists (nova_pruned_block_forward*, nova_pruned_layer_forward,
 *    nova_restore_from_cache*) first validates them on the device: cu_keep[0] = 0, 0 <= k_s <= N per
 *    segment, cu_keep[B] = M (<= M where M is only a bound), every keep_idx / prune_idx entry inside
 *    [0, N) and ascending within its segment. A list that fails returns NOVA_ERR_INVALID_ARG and
 *    launches nothing else, so a corrupt index is never dereferenced;
 *  - the stream is synchronised after every kernel launch, which pins an asynchronous CUDA error to
 *    the launch that caused it (reported by nova_device_status as NOVA_ERR_CUDA, launch number in
 *    nova_last_error).
 * Both cost host synchronisations: not for timed runs. Independently of debug mode every launching
 * call opens an NVTX range named after itself (no cost unless a tool listens). */
nova_status nova_set_debug(nova_ctx* ctx, int on);

/* ---- measurement (no counterpart in the paper) --------------------------------- */
/* Kernels launched by this context since nova_create. */
unsigned long long nova_launch_count(const nova_ctx* ctx);
/* Per-kernel timing: between nova_profile_begin and nova_profile_end every kernel launch is
 * bracketed by CUDA events on its stream. nova_profile_end waits for them and fills
 * ms[c] / launches[c] (host arrays of n >= nova_profile_categories() entries) with the summed
 * device time and the launch count of category c; nova_profile_category_name(c) names it.
 * nova_profile_select restricts the brackets to the categories whose bit is set in category_mask
 * (bit c = category c; all by default): each bracket costs two event records on the stream, which
 * shows in a step of a few hundred launches. */
int         nova_profile_categories(void);
const char* nova_profile_category_name(int cat);
nova_status nova_profile_select(nova_ctx* ctx, unsigned long long category_mask);
nova_status nova_profile_begin(nova_ctx* ctx);
nova_status nova_profile_end(nova_ctx* ctx, double* ms, long long* launches, int n);

/* ---- Eq. 4 and Eq. 7: entropy ------------------------------------------------- */
/*
 * logits: device, [S, N, V], dtype dt, row r = s*N + i starts at element r*row_stride
 *         (row_stride >= V; a multiple of 8 for bf16, 4 for f32).
 * ent:    device f32 [S, N]   ent[s,i] = -sum_v p(v) ln p(v), p = softmax(row), natural log.
 * mean:   device f32 [S] or NULL   mean[s] = (1/N) sum_i ent[s,i], summed in a fixed order.
 * A -inf logit contributes 0. A +inf or NaN logit makes the row's entropy NaN and records
 * NOVA_ERR_NONFINITE in the device status word. Negative zeros are returned as +0.
 * Errors: S,N < 0 or V < 1 -> INVALID_ARG; misaligned pointer/stride -> ALIGNMENT.
 * S*N == 0 is a no-op.
 */
nova_status nova_scale_entropy(nova_ctx* ctx, const void* logits, nova_dtype dt,
                               int S, int N, int V, int64_t row_stride,
                               float* ent, float* mean, void* stream);

/*
 * The entropy maps of all layers of a scale in one call. The layers' logits are inputs of the scale
 * (Eq. 12 takes one mean per layer), so nothing orders them behind the layers themselves: one launch
 * streams the rows of all layers, which keeps HBM busy instead of ramping up and draining per layer.
 * logits: HOST array of n_layers device pointers, each a [S, N, V] tensor as for nova_scale_entropy
 *         (same dt, V and row_stride for all). n_layers * S <= 256 for the one-launch path.
 * ent:    device f32 [n_layers, S, N].   mean: device f32 [n_layers, S] or NULL.
 * Results and errors are those of n_layers calls of nova_scale_entropy.
 */
nova_status nova_scale_entropy_layers(nova_ctx* ctx, const void* const* logits, int n_layers, nova_dtype dt,
                                      int S, int N, int V, int64_t row_stride,
                                      float* ent, float* mean, void* stream);

/* ---- Eq. 4 and Eq. 7 from the hidden states: codebook head fused with the entropy -- */
/*
 * The paper's complexity analysis (paragraph after Table 8) assumes that decoding has the
 * predicted distributions at hand anyway; a decoder that has the hidden states at hand can skip
 * writing the V-wide logits altogether. This call computes, per token,
 *   logits = x W_head^T + b_head (bf16 operands, fp32 accumulation, never rounded or stored),
 *   ent = -sum_v p(v) ln p(v), p = softmax(logits), and mean[s] = (1/N) sum_i ent[s, i].
 * x:      device bf16 [S*N, C] contiguous.   w_head: device bf16 [V, C] ([out, in] row-major).
 * b_head: device bf16 [V] or NULL.           ent: device f32 [S, N].   mean: device f32 [S] or NULL.
 * C must be a multiple of 64 and V of 32. A non-finite logit makes the row's entropy NaN and
 * records NOVA_ERR_NONFINITE in the device status word. S*N == 0 is a no-op.
 * Errors: bad sizes -> INVALID_ARG / SHAPE; misaligned pointer -> ALIGNMENT.
 */
nova_status nova_head_entropy(nova_ctx* ctx, const void* x, const void* w_head, const void* b_head,
                              int S, int N, int C, int V, float* ent, float* mean, void* stream);

/* ---- Eq. 8-13: trigger, ratios, keep counts (host arithmetic, double) ---------- */
typedef struct nova_sched_params {
    int    t_est;            /* scales kept dense to estimate the growth baseline (paper: 5) */
    double alpha;            /* Eq. 10 fraction of the baseline (paper: 0.5)                 */
    double tau;              /* Eq. 11 sigmoid temperature (paper: 0.8)                      */
    double lambda;           /* Eq. 11 weight of tanh(g_t) (paper: 0.1)                      */
    int    k_min;            /* lower bound of a keep count (default 1)                      */
    double ratio_max;        /* upper clamp of a reduction ratio (default 1)                 */
    int    force_act_scale;  /* 0: adaptive trigger; >0: fixed activation scale              */
    double force_keep_ratio; /* <0: Eq. 11-13; in [0,1]: reduction ratio = 1 - this          */
} nova_sched_params;

/* Fills *p with the paper's hyper-parameters and this library's default clamps. */
void nova_sched_params_default(nova_sched_params* p);

/*
 * All pointers are host memory. hbar_scale [B, t]: mean entropies of scales 1..t
 * (current included); hbar_layer [B, j]: mean entropies of layers 1..j of scale t
 * (may be NULL when j == 1).
 * Per image b:
 *   g_u = H_u - H_{u-1}; eta = mean(g_2..g_{t_est}); t_star[b] = first u in [t_est+1, t]
 *   with (g_u + g_{u-1})/2 <= alpha*eta, or 0; act_scale[b] = t_star+1 or 0 (Eq. 8-10).
 *   If t >= act_scale > 0: ratio_scale = sigmoid((t-act_scale)/tau) - lambda*tanh(g_t)
 *   (Eq. 11); ratio_layer = ratio_scale for j == 1, else ratio_scale - Delta*ratio_scale with
 *   Delta = (H_{t,j} - mu)/mu, mu = mean of layers 1..j-1 (mu == 0 -> Delta = 0) (Eq. 12-13).
 *   Otherwise both ratios are 0.
 *   keep[b] = N_t - floor(clamp(ratio_layer, 0, ratio_max) * N_t), clamped to [k_min, N_t].
 * Ratios are reduction ratios (fraction pruned). Errors: null pointer, B < 0, t < 1,
 * j < 1, N_t < 1, t_est < 2, tau <= 0 -> INVALID_ARG.
 */
nova_status nova_keep_ratios(const nova_sched_params* p, int B, int t, int j, int N_t,
                             const float* hbar_scale, const float* hbar_layer,
                             int32_t* t_star, int32_t* act_scale,
                             double* ratio_scale, double* ratio_layer, int32_t* keep);

/*
 * Eq. 8-13 for all L layers of scale t at once (host arithmetic, double), given the L layer means
 * of the scale: layer j's ratio uses the means of layers 1..j exactly as nova_keep_ratios(.., j, ..).
 * hbar_scale host [B, t]; hbar_layer host [B, L]; t_star, act_scale host int32 [B]; ratio_scale
 * host double [B]; ratio_layer host double [L, B]; keep host int32 [L, B]. Errors as nova_keep_ratios.
 */
nova_status nova_keep_ratios_layers(const nova_sched_params* p, int B, int t, int L, int N_t,
                                    const float* hbar_scale, const float* hbar_layer,
                                    int32_t* t_star, int32_t* act_scale,
                                    double* ratio_scale, double* ratio_layer, int32_t* keep);

/* ---- keep the highest-entropy tokens ------------------------------------------- */
/*
 * ent:  device f32 [S, N] (finite).   k: HOST int32 [S], 0 <= k[s] <= N.
 * Token i of segment s is kept iff fewer than k[s] tokens j of the segment have
 * ent[j] > ent[i] or (ent[j] == ent[i] and j < i)   (+0 and -0 compare equal).
 * keep_idx:  device int32 [sum k]        kept in-segment indices, ascending, segments concatenated
 * prune_idx: device int32 [S*N - sum k]  pruned in-segment indices, ascending, concatenated
 * cu_keep:   device int32 [S+1]          cu_keep[s] = k[0] + ... + k[s-1]
 * pos:       device int32 [S, N] or NULL position of i in its segment's kept list, -1 if pruned
 * Errors: N > 16384 -> SHAPE; k[s] outside [0, N] -> INVALID_ARG. S*N == 0 writes only cu_keep.
 */
nova_status nova_select_topk(nova_ctx* ctx, const float* ent, int S, int N, const int32_t* k,
                             int32_t* keep_idx, int32_t* prune_idx, int32_t* cu_keep,
                             int32_t* pos, void* stream);

/*
 * The selection of all layers of a scale in one launch (the pruning sentence after Eq. 13 applies
 * per layer with that layer's ratio): G lists (layers) of S segments (images) each. List g is what
 * nova_select_topk(ent + g*S*N, S, N, k + g*S, ...) gives, written to
 *   keep_idx + g*S*N, prune_idx + g*S*N (each list has room for S*N entries), cu_keep + g*(S+1),
 *   pos + g*S*N (or pos == NULL).
 * k: HOST int32 [G, S]. S <= 256. Errors as nova_select_topk. The _device form takes k from device
 * memory (clamped to [0, N]) as nova_select_topk_device does.
 */
nova_status nova_select_topk_grouped(nova_ctx* ctx, const float* ent, int G, int S, int N, const int32_t* k,
                                     int32_t* keep_idx, int32_t* prune_idx, int32_t* cu_keep,
                                     int32_t* pos, void* stream);
nova_status nova_select_topk_grouped_device(nova_ctx* ctx, const float* ent, int G, int S, int N,
                                            const int32_t* k_dev, int32_t* keep_idx, int32_t* prune_idx,
                                            int32_t* cu_keep, int32_t* pos, void* stream);

/* ---- alternative selection scores (the paper's selection-metric ablation) ------------------ */
/*
 * The ablation table on token selection metrics compares the entropy with an attention-based and an
 * MSE-based criterion; the paper names them and says only that the MSE one stands for the magnitude
 * of the frequency signal. The two calls below are this library's readings; each writes one score
 * per token, and nova_select_topk keeps the highest scores exactly as it does for entropies.
 *
 * nova_score_mse: score[b, i] = (1/C) sum_c (x[b, i, c] - U(ref_prev)[b, i, c])^2, U the bilinear
 *   resize of Eq. 16 (half-pixel centres, edge clamp) from (hp, wp) to (h, w): the energy of the
 *   detail that the previous scale's map cannot carry. x device bf16 [B, h*w, C]; ref_prev device bf16
 *   [B, hp, wp, C]; score device f32 [B, h*w]. C a multiple of 8.
 * nova_score_attention_mass: with the scale's N tokens as queries and, as keys, the kv_len[b] rows of
 *   k_cache followed by the N tokens' own keys (all tokens, nothing pruned), per head
 *   P = softmax_rows(q K^T / sqrt(dh)); score[b, j] = (1 / (n_heads * N)) sum_heads sum_queries
 *   P[query, kv_len[b] + j]: the share of the scale's attention that lands on token j's key.
 *   q, k device bf16 [B, N, C]; k_cache device bf16 [B, Lmax, C] and kv_len device int32 [B], or both
 *   NULL (no prior keys); lse_scratch device f32 [B, n_heads, N] (scratch); score device f32 [B, N].
 *   Head size 64 or 128. Sums run in a fixed order: results are reproducible bit for bit.
 * Errors: bad sizes -> INVALID_ARG / SHAPE; misaligned pointers -> ALIGNMENT. Empty inputs are no-ops.
 */
nova_status nova_score_mse(nova_ctx* ctx, const void* x, const void* ref_prev, int B, int hp, int wp,
                           int h, int w, int C, float* score, void* stream);
nova_status nova_score_attention_mass(nova_ctx* ctx, const void* q, const void* k, const void* k_cache,
                                      const int32_t* kv_len, int B, int N, int C, int n_heads, int Lmax,
                                      float* lse_scratch, float* score, void* stream);

/* ---- Eq. 14: the layer on the kept tokens -------------------------------------- */
typedef struct nova_block_weights {  /* device bf16; matrices are [out, in] row-major */
    const void *ln1_g, *ln1_b;       /* [C]            */
    const void *w_qkv, *b_qkv;       /* [3C, C], [3C]  rows 0..C-1 -> q, C..2C-1 -> k, 2C.. -> v */
    const void *w_o, *b_o;           /* [C, C], [C]    */
    const void *ln2_g, *ln2_b;       /* [C]            */
    const void *w_fc1, *b_fc1;       /* [F, C], [F]    */
    const void *w_fc2, *b_fc2;       /* [C, F], [C]    */
    float eps;                       /* LayerNorm epsilon */
} nova_block_weights;

typedef struct nova_block_shape {
    int B;        /* images                                         */
    int N;        /* tokens per image at this scale                 */
    int C;        /* width; multiple of 64                          */
    int n_heads;  /* C / n_heads must be 64 or 128                  */
    int F;        /* MLP hidden width; multiple of 64               */
    int Lmax;     /* rows per image of the K/V caches               */
    int M;        /* total kept tokens = cu_keep[B] (host knows it) */
} nova_block_shape;

/* Bytes of workspace nova_pruned_block_forward needs for this shape (0 on bad shape). */
size_t      nova_block_workspace_bytes(const nova_block_shape* s);
/* Gives the context a device buffer (256-byte aligned) used as scratch by later calls. */
nova_status nova_set_workspace(nova_ctx* ctx, void* dev_ptr, size_t bytes);

/*
 * Pre-LayerNorm transformer block on the compacted kept rows:
 *   Xc = rows keep_idx of x_in;  h = LN(Xc);  [q|k|v] = h W_qkv^T + b_qkv;
 *   keys/values of image b = k_cache[b, 0:kv_len[b]] followed by the kept tokens' own k, v;
 *   o = softmax(q K^T / sqrt(dh)) V per head (no mask);  x1 = Xc + o W_o^T + b_o;
 *   y = x1 + GELU_tanh(LN(x1) W_fc1^T + b_fc1) W_fc2^T + b_fc2.
 * x_in:     device bf16 [B, N, C]
 * keep_idx: device int32 [M], cu_keep: device int32 [B+1] (as written by nova_select_topk)
 * k_cache, v_cache: device bf16 [B, Lmax, C]; rows [0, kv_len[b]) are valid. The kept
 *           tokens' k and v are always written to rows kv_len[b] .. kv_len[b]+k_b-1
 *           (so kv_len[b] + k_b <= Lmax is required and is checked on the device:
 *           an overflowing image records NOVA_ERR_SHAPE in the device status word and
 *           its rows are not written).
 * kv_len:   device int32 [B]; if append_kv != 0 it is advanced by k_b at the end.
 * y_kept:   device bf16 [M, C], compacted order.
 * Arithmetic: bf16 operands, fp32 accumulation on the tensor cores; LayerNorm, softmax,
 * GELU and residual adds in fp32; activations between stages stored as bf16.
 * Errors: bad shape -> SHAPE; workspace smaller than nova_block_workspace_bytes ->
 * WORKSPACE; misaligned pointers -> ALIGNMENT. M == 0 is a no-op.
 */
nova_status nova_pruned_block_forward(nova_ctx* ctx, const nova_block_weights* w,
                                      const nova_block_shape* s, const void* x_in,
                                      const int32_t* keep_idx, const int32_t* cu_keep,
                                      void* k_cache, void* v_cache, int32_t* kv_len,
                                      int append_kv, void* y_kept, void* stream);

/* ---- Eq. 14 with per-image adaptive LayerNorm (class-conditional VAR backbones) ------ */
/*
 * The paper accelerates existing VAR backbones and names only the layer's two parts (attention,
 * FFN; Table 8). The class-conditional VAR models modulate each block per image from the
 * condition embedding: LayerNorm output * (1 + scale) + shift before each part and a gate on each
 * part's output. This call is nova_pruned_block_forward with those six per-image vectors:
 *   h  = LN1(Xc) * (1 + scale1[b]) + shift1[b];   x1 = Xc + gate1[b] * (attention(h) W_o^T + b_o)
 *   h2 = LN2(x1) * (1 + scale2[b]) + shift2[b];   y  = x1 + gate2[b] * (MLP(h2))
 * where b is the image of the row and LN1/LN2 keep their own affine parameters from `w` (pass
 * ones and zeros for a LayerNorm without them). Each pointer is device bf16 [B, C] or NULL (term
 * absent); mod == NULL is the plain block. m_on_device != 0 makes s->M an upper bound as in
 * nova_pruned_block_forward_device. Everything else as nova_pruned_block_forward.
 */
typedef struct nova_block_modulation {
    const void *shift1, *scale1, *gate1;   /* attention half */
    const void *shift2, *scale2, *gate2;   /* MLP half       */
} nova_block_modulation;

nova_status nova_pruned_block_forward_adaln(nova_ctx* ctx, const nova_block_weights* w,
                                            const nova_block_modulation* mod,
                                            const nova_block_shape* s, const void* x_in,
                                            const int32_t* keep_idx, const int32_t* cu_keep,
                                            void* k_cache, void* v_cache, int32_t* kv_len,
                                            int append_kv, void* y_kept, int m_on_device, void* stream);

/* ---- Eq. 14 with the parts of the text-conditioned backbones ------------------------------ */
/*
 * The text-to-image backbones the paper accelerates (Infinity) differ from the plain block in three
 * places; the paper names only the layer's parts, so the forms below are the backbones' published
 * ones. Each group is optional (NULL pointers = absent):
 *  - QK normalisation: per head, q and k are scaled to unit L2 norm, x / max(||x||, qk_eps), and
 *    multiplied by a per-channel gain; qk_gain_q, qk_gain_k device bf16 [C] (both or neither).
 *  - Rotary embedding, after the normalisation: within every head the channel pairs (2i, 2i+1) of
 *    q and k are rotated, (a, b) -> (a cos - b sin, a sin + b cos), cos and sin taken from rope_cos,
 *    rope_sin (device f32 [N, dh/2], both or neither) at the token's index in the scale, so the
 *    caller decides the position scheme (1-D, axial 2-D, ...). Keys enter the cache transformed.
 *  - Cross-attention after the self-attention residual: q2 = LN(x1; lnc_g, lnc_b) W_q2^T + b_q2
 *    attends, per head and without mask, to the cond_len[b] rows of the image's condition keys and
 *    values cond_k, cond_v (device bf16 [B, Lc_max, C], already projected by the caller);
 *    x1 <- x1 + o2 W_o2^T + b_o2. An image with cond_len 0 receives only b_o2.
 * mod (adaptive LayerNorm) and m_on_device as in nova_pruned_block_forward_adaln; everything else as
 * nova_pruned_block_forward. Errors: half-given groups -> INVALID_ARG; misaligned pointers -> ALIGNMENT.
 */
typedef struct nova_block_extras {
    const float *rope_cos, *rope_sin;
    const void *qk_gain_q, *qk_gain_k;
    float qk_eps;
    const void *lnc_g, *lnc_b, *w_q2, *b_q2, *w_o2, *b_o2;
    const void *cond_k, *cond_v;
    const int32_t* cond_len;
    int Lc_max;
} nova_block_extras;

nova_status nova_pruned_block_forward_ext(nova_ctx* ctx, const nova_block_weights* w,
                                          const nova_block_modulation* mod, const nova_block_extras* ext,
                                          const nova_block_shape* s, const void* x_in,
                                          const int32_t* keep_idx, const int32_t* cu_keep,
                                          void* k_cache, void* v_cache, int32_t* kv_len,
                                          int append_kv, void* y_kept, int m_on_device, void* stream);

/* ---- the same block for callers that cannot allocate device memory ------------------ */
/*
 * (The paper has no counterpart to this call; it exists for deployment.)
 * nova_pruned_block_forward needs a scratch buffer that the caller allocates and hands over
 * with nova_set_workspace. Some callers cannot do that: a plug-in that runs inside a host
 * program which has already given all device memory to its own pool and forbids cudaMalloc, or
 * a latency-critical serving loop where cudaMalloc/cudaFree would synchronise the whole device.
 * For them this entry point computes exactly what nova_pruned_block_forward computes, with the
 * scratch taken from a fixed array built into the library (nova_static_scratch_bytes() bytes,
 * currently 6 MiB, held by every GPU that loads the library until the process exits).
 * Arguments, layouts, results and error behaviour are those of nova_pruned_block_forward, except:
 *  - no workspace is needed or used; the context's own workspace setting is left untouched;
 *  - a shape whose nova_block_workspace_bytes() exceeds nova_static_scratch_bytes() is rejected
 *    with NOVA_ERR_WORKSPACE (nova_last_error() states both sizes). Width 1024 / MLP 4096 fits
 *    up to 256 kept rows;
 *  - the context's device must be the current CUDA device (else NOVA_ERR_INVALID_ARG);
 *  - it is refused (NOVA_ERR_INVALID_ARG) between nova_profile_begin and nova_profile_end.
 * It calls no cudaMalloc, cudaFree or other allocating routine. The first call on each device
 * looks up the array's device address (a one-time set-up); make that first call before any
 * stream capture begins. The array is shared by every call and every context in the process and
 * keeps whatever the last call left in it; the kernels never read a scratch element before
 * writing it, so nothing has to be cleared, but two calls that overlap on the GPU (different
 * streams or contexts) race on it and give undefined results: serialise them.
 */
size_t      nova_static_scratch_bytes(void);
nova_status nova_pruned_block_forward_static(nova_ctx* ctx, const nova_block_weights* w,
                                             const nova_block_shape* s, const void* x_in,
                                             const int32_t* keep_idx, const int32_t* cu_keep,
                                             void* k_cache, void* v_cache, int32_t* kv_len,
                                             int append_kv, void* y_kept, void* stream);

/* ---- Eq. 15-16: residual cache reuse -------------------------------------------- */
/*
 * x_in:       device bf16 [B, h*w, C]   layer input
 * y_kept:     device bf16 [M, C]        layer output on the kept rows (compacted)
 * keep_idx / prune_idx / cu_keep: device int32, as written by nova_select_topk (S = B, N = h*w)
 * cache_prev: device bf16 [B, hp, wp, C]  previous scale's residual cache of this layer;
 *             may be NULL only if nothing is pruned.
 * x_out:      device bf16 [B, h*w, C]:  kept rows = y_kept; pruned rows = x_in + U, where U is
 *             cache_prev resized to (h, w) bilinearly with half-pixel centres
 *             (src = (dst + 0.5) * hp / h - 0.5, clamped at the borders)            (Eq. 16)
 * cache_out:  device bf16 [B, h*w, C] or NULL:  x_out - x_in on kept rows (computed in fp32
 *             from y and x_in), U on pruned rows                                    (Eq. 15)
 * x_out must not alias x_in. C must be a multiple of 8.
 */
nova_status nova_restore_from_cache(nova_ctx* ctx, const void* x_in, const void* y_kept,
                                    const int32_t* keep_idx, const int32_t* prune_idx,
                                    const int32_t* cu_keep, const void* cache_prev,
                                    int hp, int wp, int h, int w, int C, int B, int M,
                                    void* x_out, void* cache_out, void* stream);

/* ---- Eq. 14 and Eq. 15-16 of one layer in one call ------------------------------------------ */
/*
 * nova_pruned_block_forward[_adaln] followed by nova_restore_from_cache, without the compacted
 * y_kept in between: the block's last GEMM writes each kept row straight to its place in x_out
 * (Eq. 16, kept rows) and its difference to the layer input to cache_out (Eq. 15), and the restore
 * pass then touches the pruned rows only. x_out and cache_out are bit-identical to the two calls.
 * Arguments as for those calls (mod may be NULL; cache_out may be NULL; the token map is h rows by
 * w_tokens columns, h * w_tokens == s->N;
 * m_on_device != 0: s->M is an upper bound and the kept count is cu_keep[B] on the device, and
 * cache_prev is then always required). Errors as for the two calls.
 */
nova_status nova_pruned_layer_forward(nova_ctx* ctx, const nova_block_weights* w,
                                      const nova_block_modulation* mod, const nova_block_shape* s,
                                      const void* x_in, const int32_t* keep_idx, const int32_t* prune_idx,
                                      const int32_t* cu_keep, void* k_cache, void* v_cache, int32_t* kv_len,
                                      int append_kv, const void* cache_prev, int hp, int wp, int h, int w_tokens,
                                      void* x_out, void* cache_out, int m_on_device, void* stream);

/* ---- the same steps driven from the device: no host value between the calls of a layer ----- */
/*
 * (The paper fixes what is computed, not where the keep counts live; these calls exist so that a
 * whole scale - every layer's entropy, Eq. 8-13, selection, Eq. 14 and Eq. 15-16 - can be enqueued
 * without a host synchronisation and captured once in a CUDA graph.)
 * They enqueue work only; nothing is read back. Results equal those of the host-driven calls.
 *
 * nova_keep_ratios_device: Eq. 8-13 exactly as nova_keep_ratios, one device thread per image, in
 *   double. The exp and tanh of Eq. 11 come from the device's math library instead of the host's,
 *   so a ratio may differ in its last bit; a keep count differs only if ratio * N_t lies within
 *   that bit of an integer.
 *   hbar_scale: device f32 [t, B] (row u-1 = the means of scale u, as nova_scale_entropy writes
 *   them; note the transposed layout); hbar_layer: device f32 [j, B] or NULL when j == 1;
 *   t_star, act_scale: device int32 [B] or NULL; keep: device int32 [B]. p is host memory, copied
 *   at the call.
 * nova_select_topk_device: nova_select_topk with k in device memory (int32 [S], values clamped to
 *   [0, N]); keep_idx and prune_idx must both hold S*N entries' worth of space. S <= 65535.
 * nova_pruned_block_forward_device: nova_pruned_block_forward where s->M is only an upper bound of
 *   the kept rows (it sizes launches, y_kept and the workspace: pass B*N if nothing better is
 *   known); the true count is cu_keep[B], read on the device. Rows of y_kept past it are untouched.
 * nova_restore_from_cache_device: nova_restore_from_cache with the kept count read from
 *   cu_keep[B]; cache_prev is always required (a 1 x 1 map of zeros serves before the first cache
 *   exists, when nothing can be pruned).
 * Errors as for the host-driven calls.
 */
nova_status nova_keep_ratios_device(nova_ctx* ctx, const nova_sched_params* p, int B, int t, int j, int N_t,
                                    const float* hbar_scale, const float* hbar_layer,
                                    int32_t* t_star, int32_t* act_scale, int32_t* keep, void* stream);
/* All L layers of scale t in one launch: hbar_layer device f32 [L, B] (all layers' means), keep device
 * int32 [L, B]; row j equals what nova_keep_ratios_device(.., j + 1, ..) writes. */
nova_status nova_keep_ratios_layers_device(nova_ctx* ctx, const nova_sched_params* p, int B, int t, int L, int N_t,
                                           const float* hbar_scale, const float* hbar_layer,
                                           int32_t* t_star, int32_t* act_scale, int32_t* keep, void* stream);
nova_status nova_select_topk_device(nova_ctx* ctx, const float* ent, int S, int N, const int32_t* k_dev,
                                    int32_t* keep_idx, int32_t* prune_idx, int32_t* cu_keep,
                                    int32_t* pos, void* stream);
nova_status nova_pruned_block_forward_device(nova_ctx* ctx, const nova_block_weights* w,
                                             const nova_block_shape* s, const void* x_in,
                                             const int32_t* keep_idx, const int32_t* cu_keep,
                                             void* k_cache, void* v_cache, int32_t* kv_len,
                                             int append_kv, void* y_kept, void* stream);
nova_status nova_restore_from_cache_device(nova_ctx* ctx, const void* x_in, const void* y_kept,
                                           const int32_t* keep_idx, const int32_t* prune_idx,
                                           const int32_t* cu_keep, const void* cache_prev,
                                           int hp, int wp, int h, int w, int C, int B,
                                           void* x_out, void* cache_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NOVA_H */

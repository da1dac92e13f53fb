// NOVA pruned-scale step: plain CPU oracle.
//
// TEST INFRASTRUCTURE ONLY. This file is the slow, obviously-correct statement of
// what the pruned transformer step computes. It shares no code, header, table or
// helper with the CUDA library and must never be linked, imported or called by the
// product path. Only the tests, the smoke check and the benchmark's CPU-baseline
// leg use it.
//
// Conventions: tensors are fp32 in memory (bf16 inputs are widened exactly by the
// caller), every reduction accumulates in double in index order, scalar schedule
// arithmetic is double. Loops are written as the definitions read; the only
// parallelism is an OpenMP "for" over independent rows.
//
// Every function below is pinned by CPU tests against closed forms, invariants,
// textbook special cases or brute force (nothing here is "parity unpinned").

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#include <algorithm>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

// ---------------------------------------------------------------------------
// Eq. 4 (token predictive entropy) and Eq. 7 (scale mean entropy).
//
// logits [S, N, V] row-major. For each token the predicted distribution is the
// softmax of its V logits; the entropy is -sum_v p(v) ln p(v) (natural log),
// where a term with p(v) == 0 contributes 0. mean[s] = (1/N) sum_i ent[s,i].
// ---------------------------------------------------------------------------
void oracle_scale_entropy(const float* logits, int S, int N, int V,
                          float* ent, float* mean)
{
    const long rows = (long)S * N;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        const float* z = logits + r * (long)V;
        double zmax = -INFINITY;
        for (int v = 0; v < V; ++v) zmax = std::max(zmax, (double)z[v]);
        double denom = 0.0;
        for (int v = 0; v < V; ++v) denom += std::exp((double)z[v] - zmax);
        double h = 0.0;
        for (int v = 0; v < V; ++v) {
            const double p = std::exp((double)z[v] - zmax) / denom;
            if (p > 0.0) h -= p * std::log(p);
        }
        ent[r] = (float)h;
    }
    if (mean) {
        for (int s = 0; s < S; ++s) {
            double acc = 0.0;
            for (int i = 0; i < N; ++i) acc += (double)ent[(long)s * N + i];
            mean[s] = (float)(acc / (double)N);
        }
    }
}

// ---------------------------------------------------------------------------
// Eq. 4 / Eq. 7 taken one step earlier: the predicted distribution of a token is the
// softmax of the codebook head applied to its hidden state (the paper's complexity
// paragraph after Table 8 counts the distributions as a by-product of decoding), so
//   logits[v] = sum_c x[c] * w[v, c] + b[v],   p = softmax(logits),   H = -sum p ln p.
// x [S, N, C], w [V, C] ([out, in] row-major), b [V] or null. The logits are never
// rounded: double accumulation in index order, entropy as in oracle_scale_entropy.
// ---------------------------------------------------------------------------
void oracle_head_entropy(const float* x, const float* w, const float* b, int S, int N, int C, int V,
                         float* ent, float* mean)
{
    const long rows = (long)S * N;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        const float* xr = x + r * (long)C;
        std::vector<double> z((size_t)V);
        for (int v = 0; v < V; ++v) {
            double acc = b ? (double)b[v] : 0.0;
            const float* wv = w + (long)v * C;
            for (int c = 0; c < C; ++c) acc += (double)xr[c] * (double)wv[c];
            z[v] = acc;
        }
        double zmax = -INFINITY;
        for (int v = 0; v < V; ++v) zmax = std::max(zmax, z[v]);
        double denom = 0.0;
        for (int v = 0; v < V; ++v) denom += std::exp(z[v] - zmax);
        double h = 0.0;
        for (int v = 0; v < V; ++v) {
            const double p = std::exp(z[v] - zmax) / denom;
            if (p > 0.0) h -= p * std::log(p);
        }
        ent[r] = (float)h;
    }
    if (mean) {
        for (int s = 0; s < S; ++s) {
            double acc = 0.0;
            for (int i = 0; i < N; ++i) acc += (double)ent[(long)s * N + i];
            mean[s] = (float)(acc / (double)N);
        }
    }
}

// ---------------------------------------------------------------------------
// Eq. 8-10 (growth rate, early baseline, smoothed rate, inflection scale),
// Eq. 11 (scale-linkage ratio), Eq. 12-13 (layer-linkage ratio), and the keep
// count that follows from a reduction ratio.
//
// Scales and layers are 1-based as in the paper. hbar_scale[b, u-1] is the mean
// entropy of scale u for u = 1..t (row stride t); hbar_layer[b, k-1] is the mean
// entropy seen at layer k of the current scale for k = 1..j (row stride j).
//
// Readings where the paper is silent:
//  * t_star is the first u in [t_est+1, t] with smoothed growth <= alpha*eta;
//    none -> t_star = 0, activation scale 0, nothing is pruned.
//  * scale t is pruned iff t >= t_star + 1.
//  * Ratio is the pruned fraction. It is clamped to [0, ratio_max];
//    pruned = floor(Ratio * N), keep = N - pruned, then keep >= k_min.
//  * mu == 0 in Eq. 13 -> Delta = 0.
//  * force_act_scale > 0 replaces the detected activation scale;
//    force_keep_ratio in [0,1] replaces Eq. 11-13 by Ratio = 1 - keep ratio.
// ---------------------------------------------------------------------------
struct oracle_sched_params {
    int    t_est;            // scales kept dense to estimate the baseline (paper: 5)
    double alpha;            // fraction of the baseline growth (paper: 0.5)
    double tau;              // sigmoid temperature of Eq. 11 (paper: 0.8)
    double lambda;           // weight of tanh(g_t) in Eq. 11 (paper: 0.1)
    int    k_min;            // lower bound on the kept count (default 1)
    double ratio_max;        // upper clamp of the reduction ratio (default 1)
    int    force_act_scale;  // 0 = adaptive; >0 = fixed activation scale
    double force_keep_ratio; // <0 = Eq. 11-13; otherwise keep fraction in [0,1]
};

void oracle_keep_ratios(const oracle_sched_params* p, int B, int t, int j, int N_t,
                        const float* hbar_scale, const float* hbar_layer,
                        int32_t* t_star, int32_t* act_scale,
                        double* ratio_scale, double* ratio_layer, int32_t* keep)
{
    for (int b = 0; b < B; ++b) {
        const float* H = hbar_scale + (long)b * t;   // H[u-1] = mean entropy of scale u
        auto Hbar = [&](int u) { return (double)H[u - 1]; };
        auto g = [&](int u) { return Hbar(u) - Hbar(u - 1); };           // Eq. 8, u >= 2

        // Eq. 9: eta = mean of g_2 .. g_{t_est}; Eq. 10: first t' >= t_est+1 with
        // (g_t' + g_{t'-1})/2 <= alpha * eta.
        int ts = 0;
        if (p->t_est >= 2 && t >= p->t_est + 1) {
            double eta = 0.0;
            for (int u = 2; u <= p->t_est; ++u) eta += g(u);
            eta /= (double)(p->t_est - 1);
            for (int u = p->t_est + 1; u <= t; ++u) {
                const double g_smooth = (g(u) + g(u - 1)) / 2.0;
                if (g_smooth <= p->alpha * eta) { ts = u; break; }
            }
        }
        int act = (ts > 0) ? ts + 1 : 0;
        if (p->force_act_scale > 0) { act = p->force_act_scale; ts = act - 1; }
        t_star[b] = ts;
        act_scale[b] = act;

        double r_scale = 0.0, r_layer = 0.0;
        if (act > 0 && t >= act) {
            if (p->force_keep_ratio >= 0.0) {
                r_scale = 1.0 - p->force_keep_ratio;
                r_layer = r_scale;
            } else {
                // Eq. 11
                const double g_t = (t >= 2) ? g(t) : 0.0;
                const double x = ((double)t - (double)act) / p->tau;
                r_scale = 1.0 / (1.0 + std::exp(-x)) - p->lambda * std::tanh(g_t);
                // Eq. 12-13
                if (j <= 1) {
                    r_layer = r_scale;
                } else {
                    const float* HL = hbar_layer + (long)b * j;
                    double mu = 0.0;
                    for (int k = 1; k <= j - 1; ++k) mu += (double)HL[k - 1];
                    mu /= (double)(j - 1);
                    const double delta = (mu != 0.0) ? ((double)HL[j - 1] - mu) / mu : 0.0;
                    r_layer = r_scale - delta * r_scale;
                }
            }
        }
        ratio_scale[b] = r_scale;
        ratio_layer[b] = r_layer;

        double rc = r_layer;
        if (rc < 0.0) rc = 0.0;
        if (rc > p->ratio_max) rc = p->ratio_max;
        long pruned = (long)std::floor(rc * (double)N_t);
        long k = (long)N_t - pruned;
        if (k < p->k_min) k = p->k_min;
        if (k > N_t) k = N_t;
        keep[b] = (int32_t)k;
    }
}

// ---------------------------------------------------------------------------
// Keeping the highest-entropy tokens (analysis after Eq. 3; pruning sentence
// after Eq. 13): per segment, token i has rank
//     #{ j : e_j > e_i  or  (e_j == e_i and j < i) }
// and is kept iff rank < k. Comparison is IEEE (so -0.0 == +0.0). Outputs:
// keep_idx  - kept in-segment indices, ascending, segments concatenated;
// prune_idx - pruned in-segment indices, ascending, segments concatenated;
// cu_keep[s] = sum_{s'<s} k[s'] (S+1 entries);
// pos[s,i]  = position of i within its segment's kept list, or -1 if pruned.
// ---------------------------------------------------------------------------
void oracle_select_topk(const float* ent, int S, int N, const int32_t* k,
                        int32_t* keep_idx, int32_t* prune_idx, int32_t* cu_keep,
                        int32_t* pos)
{
    cu_keep[0] = 0;
    for (int s = 0; s < S; ++s) cu_keep[s + 1] = cu_keep[s] + k[s];
    for (int s = 0; s < S; ++s) {
        const float* e = ent + (long)s * N;
        std::vector<int32_t> rank(N);
#pragma omp parallel for schedule(static)
        for (int i = 0; i < N; ++i) {
            int32_t r = 0;
            for (int jx = 0; jx < N; ++jx)
                if (e[jx] > e[i] || (e[jx] == e[i] && jx < i)) ++r;
            rank[i] = r;
        }
        int32_t nk = 0, np = 0;
        const long keep_base = cu_keep[s];
        const long prune_base = (long)s * N - cu_keep[s];
        for (int i = 0; i < N; ++i) {
            if (rank[i] < k[s]) {
                keep_idx[keep_base + nk] = i;
                if (pos) pos[(long)s * N + i] = nk;
                ++nk;
            } else {
                prune_idx[prune_base + np] = i;
                if (pos) pos[(long)s * N + i] = -1;
                ++np;
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Layer_j on the kept tokens (Eq. 14). The paper names only "Self-Attention" and
// "FFN" (latency table); the block form is this build's reading: a pre-LayerNorm
// transformer block with biases, tanh-GELU, softmax(q k^T / sqrt(dh)) without
// mask, whose keys/values are the prior-scale cache followed by the kept tokens'
// own k/v (pruned tokens skip the layer and add nothing to the cache).
//
// Weights are [out, in] row-major. x_in [B, N, C]. keep_idx/cu_keep as produced
// by the selection. k_cache/v_cache [B, Lmax, C] hold kv_len[b] valid rows.
// rows/n_rows: compacted row numbers whose outputs are wanted (NULL -> all M).
// Outputs: y [n_rows, C] (block output for those rows), k_new/v_new [M, C]
// (keys and values of every kept token, i.e. what would be appended).
// ---------------------------------------------------------------------------
struct oracle_block_weights {
    const float *ln1_g, *ln1_b, *w_qkv, *b_qkv, *w_o, *b_o;
    const float *ln2_g, *ln2_b, *w_fc1, *b_fc1, *w_fc2, *b_fc2;
    float eps;
};

static void layer_norm_row(const float* x, const float* g, const float* b, float eps,
                           int C, float* out)
{
    double mean = 0.0;
    for (int c = 0; c < C; ++c) mean += (double)x[c];
    mean /= (double)C;
    double var = 0.0;
    for (int c = 0; c < C; ++c) { const double d = (double)x[c] - mean; var += d * d; }
    var /= (double)C;
    const double rstd = 1.0 / std::sqrt(var + (double)eps);
    for (int c = 0; c < C; ++c)
        out[c] = (float)(((double)x[c] - mean) * rstd * (double)g[c] + (double)b[c]);
}

// out[o] = sum_i x[i] * W[o, i] + bias[o]
static void linear_row(const float* x, const float* W, const float* bias, int n_in,
                       int n_out, float* out)
{
    for (int o = 0; o < n_out; ++o) {
        const float* w = W + (long)o * n_in;
        double acc = 0.0;
        for (int i = 0; i < n_in; ++i) acc += (double)x[i] * (double)w[i];
        out[o] = (float)(acc + (bias ? (double)bias[o] : 0.0));
    }
}

static inline double gelu_tanh(double x)
{
    const double c = 0.7978845608028654;  // sqrt(2/pi)
    return 0.5 * x * (1.0 + std::tanh(c * (x + 0.044715 * x * x * x)));
}

// Per-image modulation of the block (adaptive LayerNorm as in the class-conditional VAR
// backbones; the NOVA paper names the layer's two parts but gives no block equations, so this
// is the backbone's published form): every array is [B, C], any of the six may be NULL.
//   h1 = LN1(x) * (1 + scale1[b]) + shift1[b]        x1 = x  + gate1[b] * (attention branch)
//   h2 = LN2(x1) * (1 + scale2[b]) + shift2[b]       y  = x1 + gate2[b] * (MLP branch)
struct oracle_block_modulation {
    const float *shift1, *scale1, *gate1, *shift2, *scale2, *gate2;
};

static void modulate_row(float* h, const float* scale, const float* shift, int b, int C)
{
    for (int c = 0; c < C; ++c) {
        double v = (double)h[c];
        if (scale) v *= 1.0 + (double)scale[(long)b * C + c];
        if (shift) v += (double)shift[(long)b * C + c];
        h[c] = (float)v;
    }
}

// Block variants of the text-conditioned backbones the paper accelerates (the Infinity models use
// rotary position embedding, query/key normalisation and cross-attention to the text tokens; the
// paper itself names only the layer's parts). Every group is optional (NULL pointers = absent):
//  * QK normalisation: per head, q and k are scaled to unit L2 norm, x / max(||x||, qk_eps), and
//    multiplied by a per-channel gain (qk_gain_q / qk_gain_k, [C]); applied first.
//  * Rotary embedding: within every head, channel pairs (2i, 2i+1) of q and k are rotated by the
//    angle whose cosine and sine are rope_cos / rope_sin [N, dh/2] at the token's index in the scale:
//    (a, b) -> (a cos - b sin, a sin + b cos). Cached keys of earlier scales were rotated when they
//    were appended; the keys returned in k_new are the transformed ones.
//  * Cross-attention after the self-attention residual: q2 = LN(x1; lnc) W_q2^T + b_q2 attends (per
//    head, softmax(q2 K^T / sqrt(dh)) V, no mask) to the cond_len[b] rows of the image's condition
//    keys / values ck, cv [B, Lc_max, C]; x1 <- x1 + o2 W_o2^T + b_o2. No normalisation or rotation there.
struct oracle_block_ext {
    const float *rope_cos, *rope_sin;
    const float *qk_gain_q, *qk_gain_k;
    float qk_eps;
    const float *lnc_g, *lnc_b, *w_q2, *b_q2, *w_o2, *b_o2;
    const float *ck, *cv;
    const int32_t* cond_len;
    int Lc_max;
};

void oracle_pruned_block_forward_ext(const oracle_block_weights* w, const oracle_block_modulation* mod,
                                     const oracle_block_ext* ext,
                                     int B, int N, int C, int n_heads, int F, int Lmax,
                                     const float* x_in, const int32_t* keep_idx,
                                     const int32_t* cu_keep,
                                     const float* k_cache, const float* v_cache,
                                     const int32_t* kv_len,
                                     const int32_t* rows, int n_rows,
                                     float* y, float* k_new, float* v_new);

void oracle_pruned_block_forward_mod(const oracle_block_weights* w, const oracle_block_modulation* mod,
                                     int B, int N, int C, int n_heads, int F, int Lmax,
                                     const float* x_in, const int32_t* keep_idx,
                                     const int32_t* cu_keep,
                                     const float* k_cache, const float* v_cache,
                                     const int32_t* kv_len,
                                     const int32_t* rows, int n_rows,
                                     float* y, float* k_new, float* v_new)
{
    oracle_pruned_block_forward_ext(w, mod, nullptr, B, N, C, n_heads, F, Lmax, x_in, keep_idx, cu_keep, k_cache,
                                    v_cache, kv_len, rows, n_rows, y, k_new, v_new);
}

// q or k of one token, all heads, in place: QK normalisation, then the rotation for position `pos`
static void qk_transform_row(float* v, const float* gain, float eps, const float* rope_cos, const float* rope_sin,
                             int pos, int n_heads, int dh)
{
    for (int hd = 0; hd < n_heads; ++hd) {
        float* h = v + hd * dh;
        if (gain) {
            double ss = 0.0;
            for (int d = 0; d < dh; ++d) ss += (double)h[d] * (double)h[d];
            const double nrm = std::max(std::sqrt(ss), (double)eps);
            for (int d = 0; d < dh; ++d) h[d] = (float)((double)h[d] / nrm * (double)gain[hd * dh + d]);
        }
        if (rope_cos) {
            for (int i = 0; i < dh / 2; ++i) {
                const double c = rope_cos[(long)pos * (dh / 2) + i], sn = rope_sin[(long)pos * (dh / 2) + i];
                const double a = h[2 * i], b = h[2 * i + 1];
                h[2 * i] = (float)(a * c - b * sn);
                h[2 * i + 1] = (float)(a * sn + b * c);
            }
        }
    }
}

void oracle_pruned_block_forward(const oracle_block_weights* w,
                                 int B, int N, int C, int n_heads, int F, int Lmax,
                                 const float* x_in, const int32_t* keep_idx,
                                 const int32_t* cu_keep,
                                 const float* k_cache, const float* v_cache,
                                 const int32_t* kv_len,
                                 const int32_t* rows, int n_rows,
                                 float* y, float* k_new, float* v_new)
{
    oracle_pruned_block_forward_mod(w, nullptr, B, N, C, n_heads, F, Lmax, x_in, keep_idx, cu_keep, k_cache,
                                    v_cache, kv_len, rows, n_rows, y, k_new, v_new);
}

void oracle_pruned_block_forward_ext(const oracle_block_weights* w, const oracle_block_modulation* mod,
                                 const oracle_block_ext* ext,
                                 int B, int N, int C, int n_heads, int F, int Lmax,
                                 const float* x_in, const int32_t* keep_idx,
                                 const int32_t* cu_keep,
                                 const float* k_cache, const float* v_cache,
                                 const int32_t* kv_len,
                                 const int32_t* rows, int n_rows,
                                 float* y, float* k_new, float* v_new)
{
    const int M = cu_keep[B];
    const int dh = C / n_heads;
    std::vector<int> seg_of(M);
    for (int b = 0; b < B; ++b)
        for (int m = cu_keep[b]; m < cu_keep[b + 1]; ++m) seg_of[m] = b;

    // gather + LN1 + k, v for every kept token
    std::vector<float> h1((size_t)M * C);
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const int b = seg_of[m];
        const float* x = x_in + ((long)b * N + keep_idx[m]) * C;
        layer_norm_row(x, w->ln1_g, w->ln1_b, w->eps, C, &h1[(size_t)m * C]);
        if (mod) modulate_row(&h1[(size_t)m * C], mod->scale1, mod->shift1, b, C);
        linear_row(&h1[(size_t)m * C], w->w_qkv + (long)C * C, w->b_qkv + C, C, C,
                   k_new + (long)m * C);
        linear_row(&h1[(size_t)m * C], w->w_qkv + 2L * C * C, w->b_qkv + 2 * C, C, C,
                   v_new + (long)m * C);
        if (ext) qk_transform_row(k_new + (long)m * C, ext->qk_gain_k, ext->qk_eps, ext->rope_cos, ext->rope_sin,
                                  keep_idx[m], n_heads, dh);
    }

    const int R = rows ? n_rows : M;
#pragma omp parallel for schedule(dynamic, 1)
    for (int ri = 0; ri < R; ++ri) {
        const int m = rows ? rows[ri] : ri;
        const int b = seg_of[m];
        const float* x = x_in + ((long)b * N + keep_idx[m]) * C;
        std::vector<float> q(C), o(C), x1(C), h2(C), f1(F), f2(C);
        linear_row(&h1[(size_t)m * C], w->w_qkv, w->b_qkv, C, C, q.data());
        if (ext) qk_transform_row(q.data(), ext->qk_gain_q, ext->qk_eps, ext->rope_cos, ext->rope_sin, keep_idx[m],
                                  n_heads, dh);

        // attention over [cache rows 0..kv_len[b]) ++ [kept rows of image b]
        const int n_old = kv_len[b];
        const int n_new = cu_keep[b + 1] - cu_keep[b];
        const int n_keys = n_old + n_new;
        std::vector<double> sc(n_keys);
        for (int hd = 0; hd < n_heads; ++hd) {
            const int c0 = hd * dh;
            auto key_row = [&](int jx) {
                return (jx < n_old) ? k_cache + ((long)b * Lmax + jx) * C + c0
                                    : k_new + ((long)cu_keep[b] + (jx - n_old)) * C + c0;
            };
            auto val_row = [&](int jx) {
                return (jx < n_old) ? v_cache + ((long)b * Lmax + jx) * C + c0
                                    : v_new + ((long)cu_keep[b] + (jx - n_old)) * C + c0;
            };
            double smax = -INFINITY;
            for (int jx = 0; jx < n_keys; ++jx) {
                const float* kr = key_row(jx);
                double acc = 0.0;
                for (int d = 0; d < dh; ++d) acc += (double)q[c0 + d] * (double)kr[d];
                sc[jx] = acc / std::sqrt((double)dh);
                smax = std::max(smax, sc[jx]);
            }
            double denom = 0.0;
            for (int jx = 0; jx < n_keys; ++jx) { sc[jx] = std::exp(sc[jx] - smax); denom += sc[jx]; }
            for (int d = 0; d < dh; ++d) {
                double acc = 0.0;
                for (int jx = 0; jx < n_keys; ++jx) acc += (sc[jx] / denom) * (double)val_row(jx)[d];
                o[c0 + d] = (float)acc;
            }
        }
        linear_row(o.data(), w->w_o, w->b_o, C, C, x1.data());
        for (int c = 0; c < C; ++c) {
            const double g1 = (mod && mod->gate1) ? (double)mod->gate1[(long)b * C + c] : 1.0;
            x1[c] = (float)((double)x[c] + g1 * (double)x1[c]);
        }

        if (ext && ext->w_q2) {
            // cross-attention to the image's condition tokens
            std::vector<float> hc(C), q2(C), o2(C), xo(C);
            layer_norm_row(x1.data(), ext->lnc_g, ext->lnc_b, w->eps, C, hc.data());
            linear_row(hc.data(), ext->w_q2, ext->b_q2, C, C, q2.data());
            const int n_c = ext->cond_len[b];
            std::vector<double> sc2(std::max(n_c, 1));
            for (int hd = 0; hd < n_heads; ++hd) {
                const int c0 = hd * dh;
                double smax = -INFINITY;
                for (int jx = 0; jx < n_c; ++jx) {
                    const float* kr = ext->ck + ((long)b * ext->Lc_max + jx) * C + c0;
                    double acc = 0.0;
                    for (int d = 0; d < dh; ++d) acc += (double)q2[c0 + d] * (double)kr[d];
                    sc2[jx] = acc / std::sqrt((double)dh);
                    smax = std::max(smax, sc2[jx]);
                }
                double denom = 0.0;
                for (int jx = 0; jx < n_c; ++jx) { sc2[jx] = std::exp(sc2[jx] - smax); denom += sc2[jx]; }
                for (int d = 0; d < dh; ++d) {
                    double acc = 0.0;
                    for (int jx = 0; jx < n_c; ++jx)
                        acc += (sc2[jx] / denom) * (double)ext->cv[((long)b * ext->Lc_max + jx) * C + c0 + d];
                    o2[c0 + d] = (float)acc;       // no condition tokens: the branch adds only its bias
                }
            }
            linear_row(o2.data(), ext->w_o2, ext->b_o2, C, C, xo.data());
            for (int c = 0; c < C; ++c) x1[c] = (float)((double)x1[c] + (double)xo[c]);
        }

        layer_norm_row(x1.data(), w->ln2_g, w->ln2_b, w->eps, C, h2.data());
        if (mod) modulate_row(h2.data(), mod->scale2, mod->shift2, b, C);
        linear_row(h2.data(), w->w_fc1, w->b_fc1, C, F, f1.data());
        for (int i = 0; i < F; ++i) f1[i] = (float)gelu_tanh((double)f1[i]);
        linear_row(f1.data(), w->w_fc2, w->b_fc2, F, C, f2.data());
        for (int c = 0; c < C; ++c) {
            const double g2 = (mod && mod->gate2) ? (double)mod->gate2[(long)b * C + c] : 1.0;
            y[(long)ri * C + c] = (float)((double)x1[c] + g2 * (double)f2[c]);
        }
    }
}

// ---------------------------------------------------------------------------
// Eq. 15-16 (residual cache and its reuse). cache_prev [B, hp, wp, C] is the
// previous scale's Cache for this layer; it is resized to (h, w) bilinearly with
// half-pixel centres: src = (dst + 0.5) * (hp / h) - 0.5, clamped below at 0, the
// upper neighbour clamped to the last row/column. Then
//   out[kept]   = y (the layer output on the kept tokens),
//   out[pruned] = in + resized cache                          (Eq. 16)
//   cache_out   = out - in                                    (Eq. 15)
// y_kept [M, C] in compacted order. cache_out may be NULL.
// ---------------------------------------------------------------------------
void oracle_restore_from_cache(const float* x_in, const float* y_kept,
                               const int32_t* keep_idx, const int32_t* prune_idx,
                               const int32_t* cu_keep,
                               const float* cache_prev, int hp, int wp,
                               int h, int w, int C, int B,
                               float* x_out, float* cache_out)
{
    const int N = h * w;
    for (int b = 0; b < B; ++b) {
        const int kb = cu_keep[b + 1] - cu_keep[b];
        for (int m = 0; m < kb; ++m) {
            const long row = (long)b * N + keep_idx[cu_keep[b] + m];
            const float* ysrc = y_kept + ((long)cu_keep[b] + m) * C;
            for (int c = 0; c < C; ++c) {
                x_out[row * C + c] = ysrc[c];
                if (cache_out) cache_out[row * C + c] = (float)((double)ysrc[c] - (double)x_in[row * C + c]);
            }
        }
        const long prune_base = (long)b * N - cu_keep[b];
        const int pb = N - kb;
#pragma omp parallel for schedule(static)
        for (int m = 0; m < pb; ++m) {
            const int i = prune_idx[prune_base + m];
            const int oy = i / w, ox = i % w;
            double sy = ((double)oy + 0.5) * ((double)hp / (double)h) - 0.5;
            double sx = ((double)ox + 0.5) * ((double)wp / (double)w) - 0.5;
            if (sy < 0.0) sy = 0.0;
            if (sx < 0.0) sx = 0.0;
            int y0 = (int)std::floor(sy), x0 = (int)std::floor(sx);
            if (y0 > hp - 1) y0 = hp - 1;
            if (x0 > wp - 1) x0 = wp - 1;
            const int y1 = std::min(y0 + 1, hp - 1), x1 = std::min(x0 + 1, wp - 1);
            const double fy = sy - (double)y0, fx = sx - (double)x0;
            const float* c00 = cache_prev + (((long)b * hp + y0) * wp + x0) * C;
            const float* c01 = cache_prev + (((long)b * hp + y0) * wp + x1) * C;
            const float* c10 = cache_prev + (((long)b * hp + y1) * wp + x0) * C;
            const float* c11 = cache_prev + (((long)b * hp + y1) * wp + x1) * C;
            const long row = (long)b * N + i;
            for (int c = 0; c < C; ++c) {
                const double top = (1.0 - fx) * (double)c00[c] + fx * (double)c01[c];
                const double bot = (1.0 - fx) * (double)c10[c] + fx * (double)c11[c];
                const double u = (1.0 - fy) * top + fy * bot;
                x_out[row * C + c] = (float)((double)x_in[row * C + c] + u);
                if (cache_out) cache_out[row * C + c] = (float)u;
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Alternative selection scores of the paper's selection-metric ablation (the table comparing
// entropy with an attention-based and an MSE-based criterion). The paper names the two criteria
// and says only that the MSE one stands for the magnitude of the frequency signal; the definitions
// below are this build's readings. Both give one score per token, and the tokens with the highest
// scores are kept by the same top-k rule as for the entropy.
//
// MSE score: how far a token's representation is from what the previous, coarser scale predicts
// for its position, i.e. the energy of the detail the coarser scale cannot carry:
//   score[b, i] = (1/C) sum_c ( x[b, i, c] - U(ref_prev)[b, i, c] )^2
// with U the bilinear resize of Eq. 16 (half-pixel centres, edge clamp) from (hp, wp) to (h, w).
// ---------------------------------------------------------------------------
void oracle_score_mse(const float* x, const float* ref_prev, int B, int hp, int wp, int h, int w, int C,
                      float* score)
{
    const int N = h * w;
    for (int b = 0; b < B; ++b) {
#pragma omp parallel for schedule(static)
        for (int i = 0; i < N; ++i) {
            const int oy = i / w, ox = i % w;
            double sy = ((double)oy + 0.5) * ((double)hp / (double)h) - 0.5;
            double sx = ((double)ox + 0.5) * ((double)wp / (double)w) - 0.5;
            if (sy < 0.0) sy = 0.0;
            if (sx < 0.0) sx = 0.0;
            int y0 = (int)std::floor(sy), x0 = (int)std::floor(sx);
            if (y0 > hp - 1) y0 = hp - 1;
            if (x0 > wp - 1) x0 = wp - 1;
            const int y1 = std::min(y0 + 1, hp - 1), x1 = std::min(x0 + 1, wp - 1);
            const double fy = sy - (double)y0, fx = sx - (double)x0;
            const float* c00 = ref_prev + (((long)b * hp + y0) * wp + x0) * C;
            const float* c01 = ref_prev + (((long)b * hp + y0) * wp + x1) * C;
            const float* c10 = ref_prev + (((long)b * hp + y1) * wp + x0) * C;
            const float* c11 = ref_prev + (((long)b * hp + y1) * wp + x1) * C;
            const float* xr = x + ((long)b * N + i) * C;
            double acc = 0.0;
            for (int c = 0; c < C; ++c) {
                const double top = (1.0 - fx) * (double)c00[c] + fx * (double)c01[c];
                const double bot = (1.0 - fx) * (double)c10[c] + fx * (double)c11[c];
                const double d = (double)xr[c] - ((1.0 - fy) * top + fy * bot);
                acc += d * d;
            }
            score[(long)b * N + i] = (float)(acc / (double)C);
        }
    }
}

// ---------------------------------------------------------------------------
// Attention-mass score: the share of the scale's attention that lands on a token's key. With the
// scale's N tokens as queries (q) and, as keys, the kv_len[b] prior-scale keys of the cache followed
// by the N tokens' own keys (k), all tokens present (nothing pruned yet), per head
//   P_h = softmax_rows( q_h K_h^T / sqrt(dh) ),        K_h = [cache rows ; k]_h
//   score[b, j] = (1 / (n_heads * N)) sum_h sum_q P_h[q, kv_len[b] + j]
// so the scores of an image sum to at most 1 (exactly 1 without prior keys).
// q, k [B, N, C]; k_cache [B, Lmax, C] (may be NULL when every kv_len is 0); score [B, N].
// ---------------------------------------------------------------------------
void oracle_score_attention_mass(const float* q, const float* k, const float* k_cache, const int32_t* kv_len,
                                 int B, int N, int C, int n_heads, int Lmax, float* score)
{
    const int dh = C / n_heads;
    for (int b = 0; b < B; ++b) {
        const int n_old = kv_len ? kv_len[b] : 0;
        const int n_keys = n_old + N;
        std::vector<double> mass((size_t)N, 0.0);
#pragma omp parallel
        {
            std::vector<double> local((size_t)N, 0.0), sc((size_t)n_keys);
#pragma omp for schedule(static) collapse(2)
            for (int hd = 0; hd < n_heads; ++hd) {
                for (int qi = 0; qi < N; ++qi) {
                    const int c0 = hd * dh;
                    const float* qr = q + ((long)b * N + qi) * C + c0;
                    double smax = -INFINITY;
                    for (int jx = 0; jx < n_keys; ++jx) {
                        const float* kr = (jx < n_old) ? k_cache + ((long)b * Lmax + jx) * C + c0
                                                       : k + ((long)b * N + (jx - n_old)) * C + c0;
                        double acc = 0.0;
                        for (int d = 0; d < dh; ++d) acc += (double)qr[d] * (double)kr[d];
                        sc[jx] = acc / std::sqrt((double)dh);
                        smax = std::max(smax, sc[jx]);
                    }
                    double denom = 0.0;
                    for (int jx = 0; jx < n_keys; ++jx) { sc[jx] = std::exp(sc[jx] - smax); denom += sc[jx]; }
                    for (int j = 0; j < N; ++j) local[j] += sc[n_old + j] / denom;
                }
            }
#pragma omp critical
            for (int j = 0; j < N; ++j) mass[j] += local[j];
        }
        for (int j = 0; j < N; ++j) score[(long)b * N + j] = (float)(mass[j] / ((double)n_heads * (double)N));
    }
}

int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

}  // extern "C"

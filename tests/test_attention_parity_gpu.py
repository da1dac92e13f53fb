"""GPU parity of the attention half of Eq. 14, measured against the attention branch itself.

The block output is y = x + attention branch + MLP branch, and with random-init weights the
residual stream x dominates it: an error metric relative to max|y| hardly sees the attention
kernel. These cases go through the ordinary nova_pruned_block_forward call with weights that
isolate the attention: W_o = I, b_o = 0, W_fc2 = 0, b_fc2 = 0, so that y = x + o with o the
concatenated heads' softmax(q K^T / sqrt(dh)) V, and with x scaled down by 2^-8 (LayerNorm
removes the scale, so q, k, v are unchanged). The metric is

    max |y_gpu - y_oracle| / max |o_oracle|,      o_oracle = y_oracle - x (gathered rows),

element-wise over the compared rows, bound by the block tolerance 2e-2. The query rows of
W_qkv are scaled up so that scores spread over several units (peaked softmax rows), K caches
get magnitude profiles that force the running maximum up between key tiles, and a query bias
against marked keys pushes their probabilities to zero. Every case states its own sensitivity
on the oracle alone: ignoring the attention branch, or half of the prior keys, moves the
metric by far more than the tolerance.
"""
import numpy as np
import pytest
import torch

import nova_synth as synth
import oracle
import paper_2602_01345_b200 as nova

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
BLOCK_TOL = 2e-2
X_SCALE = 2.0 ** -8


@pytest.fixture(scope="module")
def ctx():
    c = nova.Context(0)
    yield c
    assert c.device_status() == 0
    c.close()


def f32(t):
    return synth.to_f32_numpy(t)


def probe_weights(C, F, seed, q_gain=1.0, q_zero=False, q_bias=None, heads=1):
    """Random-init block weights with the attention branch isolated (identity output projection, no
    MLP output). q_gain scales the query rows of W_qkv (a power of two: exact in bf16); q_zero
    clears them and the query bias; q_bias puts that value on the first channel of every head's query."""
    wt = synth.block_weights(C, F, seed, DEV)
    wt["w_o"] = torch.eye(C, dtype=torch.bfloat16, device=DEV)
    wt["b_o"].zero_()
    wt["w_fc2"].zero_()
    wt["b_fc2"].zero_()
    if q_zero:
        wt["w_qkv"][:C].zero_()
        wt["b_qkv"][:C].zero_()
    else:
        wt["w_qkv"][:C] *= q_gain
    if q_bias is not None:
        dh = C // heads
        wt["b_qkv"][0:C:dh] = q_bias
    return wt


def attn_metric(y, y_ref, x_rows):
    branch = np.abs(y_ref - x_rows).max()
    return float(np.abs(y - y_ref).max() / branch), float(branch)


def attention_case(ctx, B, N, C, heads, F, Lmax, ks, kv_lens, seed, rows=None, q_gain=1.0, q_zero=False,
                   k_profile=None, dead_keys=None, half_keys_check=True, label=""):
    """Runs the block on the GPU and the oracle on the same bytes; returns the attention-branch
    error. k_profile: per-key gains [max kv_len] applied to the prior K cache. dead_keys: indices of
    prior keys that every query scores about 100 nats below the rest (query bias 16 on the first
    channel of each head, that channel of those keys set to -72 at head size 128 / -50 at 64)."""
    dh = C // heads
    wt = probe_weights(C, F, seed, q_gain=q_gain, q_zero=q_zero, q_bias=16.0 if dead_keys is not None else None,
                       heads=heads)
    x = (synth.activations(B, N, C, seed + 1, DEV).float() * X_SCALE).to(torch.bfloat16)
    k_cache, v_cache, _ = synth.kv_cache(B, Lmax, max(max(kv_lens), 1), C, seed + 2, DEV)
    if k_profile is not None:
        n = len(k_profile)
        prof = torch.tensor(np.asarray(k_profile, np.float32), device=DEV).view(1, n, 1)
        k_cache[:, :n] = (k_cache[:, :n].float() * prof).to(torch.bfloat16)
    if dead_keys is not None:
        dk = torch.as_tensor(np.asarray(dead_keys), device=DEV)
        for c0 in range(0, C, dh):
            k_cache[:, dk, c0] = -72.0 if dh == 128 else -50.0
    for b, n in enumerate(kv_lens):          # rows past each image's length must never be used
        k_cache[b, n:] = float("nan")
        v_cache[b, n:] = float("nan")
    kv_len = torch.tensor(kv_lens, dtype=torch.int32, device=DEV)
    ent = torch.rand((B, N), generator=torch.Generator(device="cpu").manual_seed(seed)).to(DEV)
    M = sum(ks)
    keep_idx = torch.empty(M, dtype=torch.int32, device=DEV)
    prune_idx = torch.empty(B * N - M, dtype=torch.int32, device=DEV)
    cu = torch.empty(B + 1, dtype=torch.int32, device=DEV)
    nova.nova_select_topk(ctx, ent, torch.tensor(ks, dtype=torch.int32), keep_idx, prune_idx, cu, None)
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, M)
    ctx.ensure_workspace(shape)
    k0, v0 = k_cache.clone(), v_cache.clone()
    y = torch.full((M, C), float("nan"), dtype=torch.bfloat16, device=DEV)
    nova.nova_pruned_block_forward(ctx, nova.BlockWeights(wt, 1e-6), shape, x, keep_idx, cu, k_cache, v_cache,
                                   kv_len, True, y)
    assert ctx.device_status() == 0

    wts = {n: f32(t) for n, t in wt.items()}
    kc, vc = np.nan_to_num(f32(k0)), np.nan_to_num(f32(v0))
    ki, cuu = keep_idx.cpu().numpy(), cu.cpu().numpy()
    rr = np.arange(M, dtype=np.int32) if rows is None else np.asarray(rows, np.int32)
    lens = np.array(kv_lens, np.int32)
    wy, _, _ = oracle.pruned_block_forward(wts, 1e-6, heads, f32(x), ki, cuu, kc, vc, lens, rows=rr)
    img = np.searchsorted(cuu, rr, side="right") - 1
    x_rows = f32(x)[img, ki[rr]]
    gy = f32(y)[rr]
    assert np.isfinite(gy).all()
    err, branch = attn_metric(gy, wy, x_rows)
    # what the metric sees, on the oracle alone: no attention branch at all ...
    dropped, _ = attn_metric(x_rows, wy, x_rows)
    assert dropped > 5 * BLOCK_TOL
    # ... and attention over only the first half of each image's prior keys
    halved = None
    if half_keys_check and max(kv_lens) >= 2:
        hy, _, _ = oracle.pruned_block_forward(wts, 1e-6, heads, f32(x), ki, cuu, kc, vc, lens // 2, rows=rr)
        touched = lens[img] >= 2
        if touched.any():
            halved, _ = attn_metric(hy[touched], wy[touched], x_rows[touched])
            assert halved > 5 * BLOCK_TOL, (label, halved)
    print(f"attention parity [{label}]: err {err:.2e} of max|o| {branch:.3f}; without attention {dropped:.2f}, "
          f"half of the prior keys {halved if halved is None else round(halved, 2)}")
    assert err <= BLOCK_TOL, (label, err)
    return err


# ------------------------------------------------------------------------------ the configurations
@pytest.mark.parametrize("q_gain", [1.0, 4.0])
def test_attention_config1_shape_dh64(ctx, q_gain):
    """Width 1024, 16 heads x 64, batch 2, 128 of 256 tokens kept over 424 prior keys, every row."""
    attention_case(ctx, B=2, N=256, C=1024, heads=16, F=4096, Lmax=680, ks=[128, 128], kv_lens=[424, 424], seed=0,
                   q_gain=q_gain, label=f"config-1 shape, query gain {q_gain}")


def test_attention_benchmark_launch(ctx):
    """The launch the benchmark times (batch 4, 2048 of 4096 kept per image, 6425 prior keys, 16 heads x
    128): 512 work items on 148 SMs, 444 whole and 68 shared by two CTAs each. Sampled rows cover the
    first and last query blocks of every image, i.e. heads on both sides of the split."""
    rows = [0, 127, 128, 255, 256, 1791, 1792, 2047, 2048, 4095, 4096, 6143, 6144, 6400, 7935, 7936, 8191]
    attention_case(ctx, B=4, N=4096, C=2048, heads=16, F=8192, Lmax=10521, ks=[2048] * 4, kv_lens=[6425] * 4, seed=19,
                   rows=rows, q_gain=4.0, half_keys_check=False, label="1024 shape, batch 4, keep 0.5")


def test_attention_all_items_key_split(ctx):
    """One image of the 1024 shape at keep ratio 0.25: 64 work items, every one shared by two CTAs whose
    partial results (different reference maxima with peaked rows) are merged."""
    rows = [0, 127, 128, 255, 256, 511, 512, 767, 768, 1023]
    attention_case(ctx, B=1, N=4096, C=2048, heads=16, F=8192, Lmax=10521, ks=[1024], kv_lens=[6425], seed=47,
                   rows=rows, q_gain=4.0, label="1024 shape, batch 1, keep 0.25")


def test_attention_2048_shape(ctx):
    """16384 tokens, 3277 kept, 26137 prior keys: 205 key tiles per work item."""
    k = 16384 - int(0.8 * 16384)
    rows = [0, 127, 128, 255, 256, 3071, 3072, 3199, 3200, k - 1]
    attention_case(ctx, B=1, N=16384, C=2048, heads=16, F=8192, Lmax=42521, ks=[k], kv_lens=[26137], seed=29,
                   rows=rows, q_gain=2.0, half_keys_check=False, label="2048 shape, keep 0.2")


def test_attention_512_shape_dh64(ctx):
    """VAR-d30 512 shape: 30 heads x 64, 1216 prior keys, ragged keep counts."""
    ks = [512, 300, 1024, 77]
    M = sum(ks)
    rows = [0, 255, 256, 511, 512, 811, 812, 1835, 1836, M - 1]
    attention_case(ctx, B=4, N=1024, C=1920, heads=30, F=7680, Lmax=2240, ks=ks, kv_lens=[1216] * 4, seed=23,
                   rows=rows, q_gain=4.0, label="512 shape")


# ------------------------------------------------------------------------------------ ragged corners
@pytest.mark.parametrize("C,heads", [(128, 2), (256, 2)])
def test_attention_small_ragged(ctx, C, heads):
    """Both head sizes: a 200-row image with no prior keys (two key tiles, one of them ragged), a
    77-row image (one query tile in use), an empty image and a 1-row image over 300 prior keys."""
    attention_case(ctx, B=4, N=200, C=C, heads=heads, F=256, Lmax=512, ks=[200, 77, 0, 1], kv_lens=[0, 130, 17, 300],
                   seed=3, q_gain=4.0, label=f"ragged, head size {C // heads}")


@pytest.mark.parametrize("C,heads", [(256, 2), (128, 2)])
def test_attention_partly_filled_query_blocks_over_many_key_tiles(ctx, C, heads):
    """Both head sizes (at 128 each query tile has its own issuing thread, at 64 one thread serves
    both): a 300-row image whose second query block has 44 rows (second tile unused), a 129-row image
    whose second tile has a single row, and a 256-row image with both tiles full, over 8 to 11 key
    tiles with ragged ends."""
    attention_case(ctx, B=3, N=320, C=C, heads=heads, F=256, Lmax=1400, ks=[300, 129, 256], kv_lens=[1000, 517, 777],
                   seed=13, q_gain=4.0, label=f"partly filled query blocks, head size {C // heads}")


def test_attention_q_zero_gives_mean_of_values(ctx):
    """Zero queries: every score is 0, the softmax is uniform, the output is the mean of all value
    rows (prior ones and the kept tokens' own)."""
    B, N, C, heads, F, Lmax = 2, 160, 256, 2, 256, 700
    ks, kv_lens = [160, 33], [391, 130]
    attention_case(ctx, B, N, C, heads, F, Lmax, ks, kv_lens, seed=61, q_zero=True, half_keys_check=True,
                   label="zero queries")


def test_attention_single_key_returns_its_value(ctx):
    """No prior keys and one kept token per image: the only key is the token's own, so o = v of that
    token exactly (softmax over one element)."""
    B, N, C, heads, F, Lmax = 3, 40, 256, 2, 256, 64
    wt = probe_weights(C, F, 71, q_gain=4.0)
    x = (synth.activations(B, N, C, 72, DEV).float() * X_SCALE).to(torch.bfloat16)
    k_cache = torch.full((B, Lmax, C), float("nan"), dtype=torch.bfloat16, device=DEV)
    v_cache = k_cache.clone()
    kv_len = torch.zeros(B, dtype=torch.int32, device=DEV)
    ent = torch.rand((B, N), generator=torch.Generator(device="cpu").manual_seed(7)).to(DEV)
    keep_idx = torch.empty(B, dtype=torch.int32, device=DEV)
    prune_idx = torch.empty(B * N - B, dtype=torch.int32, device=DEV)
    cu = torch.empty(B + 1, dtype=torch.int32, device=DEV)
    nova.nova_select_topk(ctx, ent, torch.ones(B, dtype=torch.int32), keep_idx, prune_idx, cu, None)
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, B)
    ctx.ensure_workspace(shape)
    y = torch.empty((B, C), dtype=torch.bfloat16, device=DEV)
    nova.nova_pruned_block_forward(ctx, nova.BlockWeights(wt, 1e-6), shape, x, keep_idx, cu, k_cache, v_cache, kv_len,
                                   True, y)
    assert ctx.device_status() == 0
    ki = keep_idx.cpu().numpy()
    x_rows = f32(x)[np.arange(B), ki]
    v_own = f32(v_cache)[:, 0]                          # the value row each image appended
    assert np.isfinite(v_own).all()
    # y = bf16(x + v): one rounding of a sum of two bf16 numbers
    want = (torch.from_numpy(x_rows + v_own)).to(torch.bfloat16).float().numpy()
    assert np.array_equal(f32(y), want)
    wy, _, wv = oracle.pruned_block_forward({n: f32(t) for n, t in wt.items()}, 1e-6, heads, f32(x), ki,
                                            cu.cpu().numpy(), np.zeros((B, Lmax, C), np.float32),
                                            np.zeros((B, Lmax, C), np.float32), np.zeros(B, np.int32))
    assert np.allclose(wy - x_rows, wv, atol=1e-6)      # the oracle agrees: o is the token's own v
    err, _ = attn_metric(f32(y), wy, x_rows)
    assert err <= BLOCK_TOL


# ----------------------------------------------------------------- peaked rows: rescale, clamp, merge
def _step_profile(n, lo=0.25, hi=4.0, at=None):
    at = n // 2 if at is None else at
    return np.r_[np.full(at, lo), np.full(n - at, hi)].astype(np.float32)


@pytest.mark.parametrize("C,heads", [(256, 2), (128, 2)])
@pytest.mark.parametrize("hi", [4.0, 8.0])
def test_attention_running_maximum_rises_across_key_tiles(ctx, C, heads, hi):
    """The prior keys' magnitude steps from 0.25 to `hi` half way through, so each row's largest
    score rises between key tiles: by roughly 9 nats (13 in log2 units) at 4, which the streaming
    softmax must carry against the reference maximum of the first key tile, and by 20 to 30 nats
    (about 2^30 to 2^45) at 8, which for some rows of every warp exceeds what is carried (2^40): the
    reference is raised and the accumulated output and row sum are rescaled in tensor memory, by
    nearly zero for those rows and by moderate factors for the other rows of the warp. 1500 prior
    keys = 12 key tiles per item, whole items (B such that the wave is not split)."""
    attention_case(ctx, B=2, N=300, C=C, heads=heads, F=256, Lmax=2000, ks=[300, 129], kv_lens=[1500, 1500], seed=83,
                   k_profile=_step_profile(1500, hi=hi), label=f"rising maximum to x{hi}, head size {C // heads}")


def test_attention_rising_maximum_in_key_split_items(ctx):
    """Four work items on 148 SMs: each is shared by two CTAs, one per half of the keys. With the
    magnitude step at the middle, the two halves finish with reference maxima many units apart, so
    the merge weights of the low half underflow towards zero."""
    attention_case(ctx, B=1, N=600, C=256, heads=2, F=2048, Lmax=1024, ks=[300], kv_lens=[517], seed=53,
                   k_profile=_step_profile(517, at=384, hi=8.0), label="rising maximum, key-split items")


@pytest.mark.parametrize("C,heads", [(256, 2), (128, 2)])
def test_attention_keys_with_vanishing_probability(ctx, C, heads):
    """Every fourth prior key scores about 100 nats below the others for every query (a query bias
    against a marked key channel): their probabilities are exactly 0 in the oracle and must contribute
    nothing on the GPU either (flushed by the special-function unit, clamped at 2^-126 by the polynomial)."""
    dead = np.arange(0, 900, 4)
    attention_case(ctx, B=2, N=300, C=C, heads=heads, F=256, Lmax=1400, ks=[300, 77], kv_lens=[900, 900], seed=89,
                   q_gain=2.0, dead_keys=dead, label=f"vanishing probabilities, head size {C // heads}")


# ------------------------------------------------- block variants: rotary embedding, QK norm, cross-attention
def _rope_tables(h, w, dh, seed):
    """Axial 2-D rotary tables for an h x w token grid: the first half of a head's channel pairs turns
    with the row index, the second half with the column index, at geometrically spaced frequencies."""
    n_pairs = dh // 2
    half = n_pairs // 2
    freq = 1.0 / (100.0 ** (torch.arange(half, dtype=torch.float64) / half))
    ys, xs = torch.meshgrid(torch.arange(h, dtype=torch.float64), torch.arange(w, dtype=torch.float64), indexing="ij")
    ang = torch.cat([ys.reshape(-1, 1) * freq, xs.reshape(-1, 1) * freq], dim=1)          # [N, dh/2]
    return torch.cos(ang).float().to(DEV), torch.sin(ang).float().to(DEV)


@pytest.mark.parametrize("parts", ["rope", "qk_norm", "cross", "all", "all_modulated_device_count"])
@pytest.mark.parametrize("C,heads", [(256, 2), (256, 4)])
def test_block_variants_match_oracle(ctx, parts, C, heads):
    """Rotary embedding, QK normalisation and cross-attention (one at a time and together, also with
    adaptive-LayerNorm modulation and the kept count left on the device) against the oracle, with the
    attention branches isolated (identity output projections, no MLP output, small input): the error is
    taken relative to the attention output, and the transformed keys appended to the cache are compared too."""
    B, h, w, F, Lmax, Lc = 3, 12, 15, 256, 700, 40
    N, dh = h * w, C // heads
    ks, kv_lens, cond_lens = [180, 77, 5], [300, 130, 0], [40, 7, 0]
    seed = 91
    wt = probe_weights(C, F, seed, q_gain=1.0 if "qk" in parts or parts.startswith("all") else 4.0)
    x = (synth.activations(B, N, C, seed + 1, DEV).float() * X_SCALE).to(torch.bfloat16)
    k_cache, v_cache, _ = synth.kv_cache(B, Lmax, max(kv_lens), C, seed + 2, DEV)
    use_rope = parts in ("rope", "all", "all_modulated_device_count")
    use_norm = parts in ("qk_norm", "all", "all_modulated_device_count")
    use_cross = parts in ("cross", "all", "all_modulated_device_count")
    ext = {}
    g = torch.Generator(device="cpu").manual_seed(seed)
    if use_norm:
        # unit-norm heads of random directions are nearly orthogonal: a large query gain spreads the scores
        ext["qk_gain_q"] = (256.0 * (1 + 0.1 * torch.randn(C, generator=g))).to(torch.bfloat16).to(DEV)
        ext["qk_gain_k"] = (1 + 0.1 * torch.randn(C, generator=g)).to(torch.bfloat16).to(DEV)
        # prior keys as the cache holds them under this variant: unit heads
        kc = k_cache.float().view(B, Lmax, heads, dh)
        k_cache = (kc / kc.norm(dim=-1, keepdim=True).clamp_min(1e-6)).view(B, Lmax, C).to(torch.bfloat16)
    if use_rope:
        ext["rope_cos"], ext["rope_sin"] = _rope_tables(h, w, dh, seed)
    if use_cross:
        ext["lnc_g"] = synth.randn_bf16((C,), seed + 3, DEV, std=0.02, mean=1.0)
        ext["lnc_b"] = synth.randn_bf16((C,), seed + 4, DEV, std=0.02)
        ext["w_q2"] = synth.randn_bf16((C, C), seed + 5, DEV, std=0.08)
        ext["b_q2"] = synth.randn_bf16((C,), seed + 6, DEV, std=0.02)
        ext["w_o2"] = torch.eye(C, dtype=torch.bfloat16, device=DEV)
        ext["b_o2"] = torch.zeros(C, dtype=torch.bfloat16, device=DEV)
        ext["cond_k"] = synth.randn_bf16((B, Lc, C), seed + 7, DEV)
        ext["cond_v"] = synth.randn_bf16((B, Lc, C), seed + 8, DEV)
        for b, n in enumerate(cond_lens):
            ext["cond_k"][b, n:] = float("nan")
            ext["cond_v"][b, n:] = float("nan")
        ext["cond_len"] = torch.tensor(cond_lens, dtype=torch.int32, device=DEV)
    md = None
    on_device = parts == "all_modulated_device_count"
    if on_device:
        md = {n: (0.3 * torch.randn((B, C), generator=g)).to(torch.bfloat16).to(DEV) for n in nova.MODULATION_NAMES}
    for b, n in enumerate(kv_lens):
        k_cache[b, n:] = float("nan")
        v_cache[b, n:] = float("nan")
    kv_len = torch.tensor(kv_lens, dtype=torch.int32, device=DEV)
    ent = torch.rand((B, N), generator=torch.Generator(device="cpu").manual_seed(seed)).to(DEV)
    M = sum(ks)
    cap = B * N if on_device else M
    keep_idx = torch.zeros(cap, dtype=torch.int32, device=DEV)
    prune_idx = torch.empty(B * N - M, dtype=torch.int32, device=DEV)
    cu = torch.empty(B + 1, dtype=torch.int32, device=DEV)
    nova.nova_select_topk(ctx, ent, torch.tensor(ks, dtype=torch.int32), keep_idx[:M], prune_idx, cu, None)
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, cap)
    ctx.ensure_workspace(shape)
    k0, v0 = k_cache.clone(), v_cache.clone()
    y = torch.full((cap, C), float("nan"), dtype=torch.bfloat16, device=DEV)
    nova.nova_pruned_block_forward_ext(ctx, nova.BlockWeights(wt, 1e-6), md, ext, shape, x, keep_idx, cu, k_cache, v_cache,
                                       kv_len, True, y, m_on_device=on_device)
    assert ctx.device_status() == 0

    wts = {n: f32(t) for n, t in wt.items()}
    oext = {}
    for n, t in ext.items():
        name = {"cond_k": "ck", "cond_v": "cv"}.get(n, n)
        oext[name] = t.cpu().numpy() if n == "cond_len" else np.nan_to_num(f32(t))
    ki, cuu = keep_idx[:M].cpu().numpy(), cu.cpu().numpy()
    lens = np.array(kv_lens, np.int32)
    mod_np = {n: f32(t) for n, t in md.items()} if md else None
    wy, wk, _ = oracle.pruned_block_forward_ext(wts, 1e-6, heads, f32(x), ki, cuu, np.nan_to_num(f32(k0)),
                                                np.nan_to_num(f32(v0)), lens, oext, modulation=mod_np)
    img = np.searchsorted(cuu, np.arange(M), side="right") - 1
    x_rows = f32(x)[img, ki]
    gy = f32(y)[:M]
    assert np.isfinite(gy).all()
    err, branch = attn_metric(gy, wy, x_rows)
    # the variant acts: the plain block's output is far from it in the same metric
    py, _, _ = oracle.pruned_block_forward(wts, 1e-6, heads, f32(x), ki, cuu, np.nan_to_num(f32(k0)), np.nan_to_num(f32(v0)),
                                           lens, modulation=mod_np)
    plain, _ = attn_metric(py, wy, x_rows)
    print(f"block variant [{parts}, head size {dh}]: err {err:.2e} of max|branches| {branch:.3f}; plain block {plain:.2f}")
    assert plain > 5 * BLOCK_TOL
    assert err <= BLOCK_TOL
    gk = f32(k_cache)
    for b in range(B):
        n0, kb = kv_lens[b], ks[b]
        want_rows = wk[cuu[b]:cuu[b + 1]]
        assert np.abs(gk[b, n0:n0 + kb] - want_rows).max() <= BLOCK_TOL * np.abs(want_rows).max()
    if on_device:
        assert torch.isnan(y[M:].float()).all()
    assert kv_len.cpu().tolist() == [a + b for a, b in zip(kv_lens, ks)]

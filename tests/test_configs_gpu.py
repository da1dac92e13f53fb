"""The pipeline configurations as stated: whole generations through MultiScaleRunner.

  * VAR-d16 256x256: 16 layers, width 1024, 16 heads, scales 1,2,3,4,5,6,8,10,13,16, batch 8,
    mean entropy per scale following a seeded sigmoid per image, layer-linked ratios over all 16
    layers, nothing forced: the inflection test of Eq. 8-10 fires at a seed-determined scale.
  * VAR-d30 512x512: 30 layers, width 1920, 30 heads x 64, scales 1,2,3,4,6,9,13,18,24,32, batch 4,
    seeded spatial entropy fields per scale, pruning from the detected inflection scale onward.

Decisions (inflection scale, activation scale, every keep count, every index list of every layer,
image and scale) are compared exactly with the oracle's on the entropies the GPU measured. Values
are compared layer by layer, teacher-forced (the oracle's block and restore run on the inputs the
GPU's layer had), on the last scales and on sampled layers and rows, which bounds the oracle's time.
"""
import numpy as np
import pytest
import torch

import nova_synth as synth
import oracle
import paper_2602_01345_b200 as nova
from paper_2602_01345_b200 import pipeline

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
ENT_TOL = 1e-3
BLOCK_TOL = 2e-2


def f32(t):
    return synth.to_f32_numpy(t)


def _rel_err(got, want):
    return float(np.abs(got - want).max() / np.abs(want).max())


def _bf16_ulp_ok(got, want):
    mag = np.maximum(np.abs(got), np.abs(want))
    return (np.abs(got - want) <= mag * 2.0 ** -7 + 4e-6).all()


def _generation(cfg, B, seed, spatial, fused, value_scales, value_layers, n_rows=24):
    ms = synth.CONFIGS[cfg]
    L, T, C = ms.L, len(ms.scales), ms.C
    ctx = nova.Context(0)
    weights = [synth.block_weights(C, ms.F, 1000 * seed + j, DEV) for j in range(L)]
    wts = {j: {n: f32(v) for n, v in weights[j].items()} for j in value_layers}
    gen = pipeline.MultiScaleRunner(ctx, weights, ms.heads, B, ms.scales, fused_restore=fused)
    a_env, _ = synth.scale_envelope_temperatures(B, T, seed=seed)
    beta = synth.layer_inverse_temperatures(L, seed)
    sched, osched = nova.SchedParams(), oracle.SchedParams()
    pruned_layers = checked = 0
    first_pruned_scale = None
    for t in range(1, T + 1):
        side = ms.scales[t - 1]
        N = side * side
        x_in = synth.activations(B, N, C, 200 * seed + t, DEV)
        if spatial and side >= 3:
            # a seeded smooth field per scale (from 3 x 3 tokens up), scaled by the image's envelope
            field = synth.smooth_temperature_field(B, side, side, seed * 31 + t, a_lo=0.6, a_hi=1.4, device=DEV)
            a = field * a_env[:, t - 1].view(B, 1).to(DEV)
        else:
            a = a_env[:, t - 1].view(B, 1).expand(B, N).contiguous().to(DEV)
        scale_logits = synth.logits_from_temperature(a, synth.V_CODEBOOK, 300 * seed + t)
        layer_logits = [synth.logits_from_temperature(a * float(beta[j]), synth.V_CODEBOOK, 400 * seed + 40 * t + j)
                        for j in range(L)]
        snaps = {}

        def hook(stage, j, info, t=t, snaps=snaps):
            if t not in value_scales or j not in value_layers:
                return
            if stage == "before":
                snaps[j] = dict(x_in=info["x_in"].clone(), k=info["k_cache"].clone(), v=info["v_cache"].clone(),
                                kv_len=info["kv_len"].clone(),
                                cache_prev=None if info["cache_prev"] is None else info["cache_prev"].clone())
            else:
                snaps[j].update(x_out=info["x_out"].clone(), cache_out=info["cache_out"].clone())

        x_out, keeps, runner = gen.run_scale(t, x_in, scale_logits, layer_logits, sched, layer_hook=hook)
        assert ctx.device_status() == 0
        hist = gen.hbar_scale.numpy()
        _, w_mean = oracle.scale_entropy(f32(scale_logits))
        assert np.abs(hist[:, t - 1] - w_mean).max() <= ENT_TOL
        # ---- decisions of every layer, exactly, on the GPU's own entropies
        ent_gpu = runner.ent.cpu().numpy()
        hbar_layer = runner.mean.cpu().numpy().T.copy()                       # [B, L]
        kk, pp, cc = runner.keep_idx.cpu().numpy(), runner.prune_idx.cpu().numpy(), runner.cu_keep.cpu().numpy()
        lists = {}
        for j in range(L):
            wr = oracle.keep_ratios(osched, t, j + 1, N, hist.copy(), hbar_layer[:, : j + 1].copy())
            assert np.array_equal(keeps[j].numpy(), wr["keep"]), (t, j)
            w_keep, w_prune, w_cu, _ = oracle.select_topk(ent_gpu[j], wr["keep"])
            M = int(w_cu[-1])
            assert np.array_equal(cc[j], w_cu), (t, j)
            assert np.array_equal(kk[j, :M], w_keep) and np.array_equal(pp[j, : B * N - M], w_prune), (t, j)
            lists[j] = (w_keep, w_prune, w_cu)
            if (wr["keep"] < N).any():
                pruned_layers += 1
                first_pruned_scale = first_pruned_scale or t
            # pruning happens from the activation scale onward and never before it
            assert ((wr["keep"] < N) <= ((wr["act_scale"] > 0) & (wr["act_scale"] <= t))).all()
        # ---- values, teacher-forced per layer
        for j, sn in snaps.items():
            w_keep, w_prune, w_cu = lists[j]
            M = int(w_cu[-1])
            rng = np.random.default_rng(seed * 97 + t * 13 + j)
            rows = np.unique(np.r_[0, M - 1, rng.integers(0, M, n_rows)]).astype(np.int32)
            lens = sn["kv_len"].cpu().numpy()
            wy, _, _ = oracle.pruned_block_forward(wts[j], 1e-6, ms.heads, f32(sn["x_in"]), w_keep, w_cu, f32(sn["k"]),
                                                   f32(sn["v"]), lens, rows=rows)
            gx, gc = f32(sn["x_out"]), f32(sn["cache_out"])
            img = np.searchsorted(w_cu, rows, side="right") - 1
            assert _rel_err(gx[img, w_keep[rows]], wy) <= BLOCK_TOL, (t, j)
            # the restore step on the GPU's own block output (the kept rows of x_out)
            all_rows = np.arange(M)
            img_all = np.searchsorted(w_cu, all_rows, side="right") - 1
            y_gpu = gx[img_all, w_keep]
            prev = f32(sn["cache_prev"]) if sn["cache_prev"] is not None else np.zeros((B, 1, 1, C), np.float32)
            wx, wc = oracle.restore_from_cache(f32(sn["x_in"]), y_gpu, w_keep, w_prune, w_cu, prev, side, side)
            assert _bf16_ulp_ok(gx, wx) and _bf16_ulp_ok(gc, wc), (t, j)
            checked += 1
    final = oracle.keep_ratios(osched, T, 1, ms.scales[-1] ** 2, gen.hbar_scale.numpy())
    ctx.close()
    return dict(act_scale=final["act_scale"], t_star=final["t_star"], pruned_layers=pruned_layers, checked=checked,
                first_pruned_scale=first_pruned_scale)


@pytest.mark.parametrize("fused", [False, True])
def test_var_d16_256_generation_as_configured(fused):
    """16 layers, batch 8, ten scales, the paper's hyper-parameters, nothing forced."""
    cfg = synth.CONFIGS["c2_var_d16_256"]
    assert cfg.L == 16 and cfg.B == 8
    r = _generation("c2_var_d16_256", B=cfg.B, seed=3, spatial=False, fused=fused, value_scales=(9, 10),
                    value_layers=(0, 7, 15))
    assert (r["act_scale"] > 0).any() and (r["act_scale"] <= 10).any()       # the trigger fired in time for some images
    assert len(set(r["act_scale"].tolist())) > 1                              # and at image-dependent scales
    assert r["pruned_layers"] >= 16 and r["checked"] == 6


def test_var_d30_512_generation_from_detected_inflection():
    """30 layers, width 1920, 30 heads x 64, batch 4, spatial entropy fields per scale; pruning starts
    at the scale after the detected inflection."""
    cfg = synth.CONFIGS["c3_var_d30_512"]
    assert cfg.L == 30 and cfg.B == 4
    r = _generation("c3_var_d30_512", B=cfg.B, seed=5, spatial=True, fused=True, value_scales=(10,),
                    value_layers=(0, 29), n_rows=12)
    assert (r["act_scale"] > 0).any()
    fired = r["act_scale"][r["act_scale"] > 0]
    assert r["first_pruned_scale"] == int(fired.min())                        # pruning begins exactly there
    assert r["pruned_layers"] >= 30 and r["checked"] == 2


@pytest.mark.parametrize("cfg,B,keep", [("c4_1024", 1, 0.25), ("c4_1024", 1, 0.5), ("c4_1024", 1, 0.75),
                                        ("c4_1024", 4, 0.25), ("c4_1024", 4, 0.5), ("c4_1024", 4, 0.75),
                                        ("c5_2048", 1, 0.2)])
def test_large_shapes_keep_sweep_through_the_runner(cfg, B, keep):
    """The 1024x1024 shape at keep ratios 0.25 / 0.5 / 0.75 and batch 1 / 4, and the 2048x2048 shape at
    keep 0.2: the last scale through the scale runner (two layers resident: the launch shapes are
    those of the full model), forced activation and keep ratio as the configurations state. Keep
    counts and index lists of both layers exact; the second layer's block and restore against the
    oracle on the layer's actual inputs (sampled kept rows, every pruned row)."""
    ms = synth.CONFIGS[cfg]
    L, t = 2, len(ms.scales)
    side, prev = ms.scales[-1], ms.scales[-2]
    N, P, Lmax, C = side * side, ms.prior_tokens(t), ms.total_tokens, ms.C
    ctx = nova.Context(0)
    weights = [synth.block_weights(C, ms.F, 70 + j, DEV) for j in range(L)]
    k_caches, v_caches = [], []
    for j in range(L):
        k, v, _ = synth.kv_cache(B, Lmax, P, C, 80 + 2 * j, DEV)
        k_caches.append(k)
        v_caches.append(v)
    kv_len = torch.full((L, B), P, dtype=torch.int32, device=DEV)
    cache_prev = [synth.residual_cache(B, prev, prev, C, 90 + j, DEV) for j in range(L)]
    if cfg == "c5_2048":
        a = synth.blob_temperature_field(B, side, side, 7, cover=0.2, device=DEV)      # high entropy in blobs covering 20 %
    else:
        a = synth.smooth_temperature_field(B, side, side, 7, device=DEV)
    beta = synth.layer_inverse_temperatures(L, 7)
    logits = [synth.logits_from_temperature(a * float(beta[j]), synth.V_CODEBOOK, 100 + j) for j in range(L)]
    x_in = synth.activations(B, N, C, 110, DEV)
    sched = nova.SchedParams(force_act_scale=t, force_keep_ratio=keep)
    osched = oracle.SchedParams(force_act_scale=t, force_keep_ratio=keep)
    hbar = torch.linspace(2.0, 7.0, t).repeat(B, 1).contiguous()
    runner = pipeline.PrunedScaleRunner(ctx, weights, ms.heads, B, side, side, Lmax, k_caches, v_caches, kv_len,
                                        cache_prev, fused_restore=True)
    snap = {}

    def hook(stage, j, info):
        if j != L - 1:
            return
        if stage == "before":
            snap.update(x_in=info["x_in"].clone(), k=info["k_cache"].clone(), v=info["v_cache"].clone())
        else:
            snap.update(x_out=info["x_out"].clone(), cache_out=info["cache_out"].clone())

    x_out, keeps = runner.run_scale(x_in, logits, sched, t, hbar, layer_hook=hook)
    assert ctx.device_status() == 0
    k_want = N - int((1.0 - keep) * N)
    ent_gpu = runner.ent.cpu().numpy()
    kk, pp, cc = runner.keep_idx.cpu().numpy(), runner.prune_idx.cpu().numpy(), runner.cu_keep.cpu().numpy()
    for j in range(L):
        wr = oracle.keep_ratios(osched, t, j + 1, N, hbar.numpy())
        assert np.array_equal(keeps[j].numpy(), wr["keep"]) and (wr["keep"] == k_want).all()
        w_keep, w_prune, w_cu, _ = oracle.select_topk(ent_gpu[j], wr["keep"])
        M = int(w_cu[-1])
        assert np.array_equal(cc[j], w_cu) and np.array_equal(kk[j, :M], w_keep)
        assert np.array_equal(pp[j, : B * N - M], w_prune)
    if cfg == "c5_2048":
        # the kept tokens are the high-entropy blobs: almost all of them lie where the field is hot
        hot = (a[0].cpu().numpy() < 1.0)
        assert hot[w_keep].mean() > 0.9
    j = L - 1
    rng = np.random.default_rng(3)
    rows = np.unique(np.r_[0, M - 1, rng.integers(0, M, 10)]).astype(np.int32)
    wy, _, _ = oracle.pruned_block_forward({n: f32(v) for n, v in weights[j].items()}, 1e-6, ms.heads, f32(snap["x_in"]),
                                           w_keep, w_cu, f32(snap["k"]), f32(snap["v"]), np.full(B, P, np.int32), rows=rows)
    gx, gc = f32(snap["x_out"]), f32(snap["cache_out"])
    img = np.searchsorted(w_cu, rows, side="right") - 1
    assert _rel_err(gx[img, w_keep[rows]], wy) <= BLOCK_TOL
    img_all = np.searchsorted(w_cu, np.arange(M), side="right") - 1
    wx, wc = oracle.restore_from_cache(f32(snap["x_in"]), gx[img_all, w_keep], w_keep, w_prune, w_cu, f32(cache_prev[j]),
                                       side, side)
    assert _bf16_ulp_ok(gx, wx) and _bf16_ulp_ok(gc, wc)
    assert kv_len.cpu().tolist() == [[P + k_want] * B] * L
    ctx.close()

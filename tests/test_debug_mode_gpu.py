"""Debug mode, guard bands and the selection of profiled kernel categories.

Debug mode (nova_set_debug): index lists are validated on the device before any kernel uses them,
so a corrupt list comes back as NOVA_ERR_INVALID_ARG with nothing dereferenced, and every launch is
synchronised. Results in debug mode equal the ordinary ones bit for bit.

Guard bands: every output buffer of the path sits between two pattern-filled bands that must come
back untouched, and inputs must come back unchanged, at a ragged shape that ends inside a tile in
every dimension.
"""
import numpy as np
import pytest
import torch

import nova_synth as synth
import oracle
import paper_2602_01345_b200 as nova

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
BAND_BYTES = 4096
PATTERN = 0xA5


class Banded:
    """A tensor of `shape` between two guard bands inside one allocation."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) if len(shape) else 1
        esz = torch.empty((), dtype=dtype).element_size()
        band = BAND_BYTES // esz
        self.raw = torch.empty(n + 2 * band, dtype=dtype, device=DEV)
        self.raw.view(torch.uint8).fill_(PATTERN)
        self.t = self.raw[band:band + n].view(shape)
        if fill is not None:
            self.t.fill_(fill)

    def intact(self) -> bool:
        b = self.raw.view(torch.uint8)
        return bool((b[:BAND_BYTES] == PATTERN).all()) and bool((b[-BAND_BYTES:] == PATTERN).all())


@pytest.fixture()
def ctx():
    c = nova.Context(0)
    yield c
    c.set_debug(False)
    assert c.device_status() == 0
    c.close()


def _case(seed=5):
    B, h, w, hp, wp, C, heads, F, Lmax = 3, 10, 15, 7, 9, 128, 2, 256, 512
    ks, kv_lens = [150, 37, 0], [0, 130, 17]
    N = h * w
    wt = synth.block_weights(C, F, seed, DEV)
    x = synth.activations(B, N, C, seed + 1, DEV)
    k_cache, v_cache, _ = synth.kv_cache(B, Lmax, max(kv_lens), C, seed + 2, DEV)
    cache_prev = synth.residual_cache(B, hp, wp, C, seed + 3, DEV)
    ent = torch.rand((B, N), generator=torch.Generator(device="cpu").manual_seed(seed)).to(DEV)
    return dict(B=B, h=h, w=w, hp=hp, wp=wp, C=C, heads=heads, F=F, Lmax=Lmax, ks=ks, kv_lens=kv_lens, N=N,
                wt=wt, x=x, k_cache=k_cache, v_cache=v_cache, cache_prev=cache_prev, ent=ent)


def _lists(ctx, c):
    B, N, M = c["B"], c["N"], sum(c["ks"])
    keep_idx = torch.empty(M, dtype=torch.int32, device=DEV)
    prune_idx = torch.empty(B * N - M, dtype=torch.int32, device=DEV)
    cu = torch.empty(B + 1, dtype=torch.int32, device=DEV)
    nova.nova_select_topk(ctx, c["ent"], torch.tensor(c["ks"], dtype=torch.int32), keep_idx, prune_idx, cu, None)
    return keep_idx, prune_idx, cu


def _layer(ctx, c, keep_idx, prune_idx, cu):
    B, N, C = c["B"], c["N"], c["C"]
    shape = nova.BlockShape(B, N, C, c["heads"], c["F"], c["Lmax"], sum(c["ks"]))
    ctx.ensure_workspace(shape)
    kc, vc = c["k_cache"].clone(), c["v_cache"].clone()
    kv_len = torch.tensor(c["kv_lens"], dtype=torch.int32, device=DEV)
    x_out = torch.full_like(c["x"], float("nan"))
    cache_out = torch.full_like(c["x"], float("nan"))
    nova.nova_pruned_layer_forward(ctx, nova.BlockWeights(c["wt"], 1e-6), None, shape, c["x"], keep_idx, prune_idx, cu,
                                   kc, vc, kv_len, True, c["cache_prev"], c["h"], c["w"], x_out, cache_out)
    return x_out, cache_out, kc, vc, kv_len


def test_debug_mode_gives_the_same_results(ctx):
    c = _case()
    keep_idx, prune_idx, cu = _lists(ctx, c)
    plain = _layer(ctx, c, keep_idx, prune_idx, cu)
    ctx.set_debug(True)
    checked = _layer(ctx, c, keep_idx, prune_idx, cu)
    assert ctx.device_status() == 0
    for a, b in zip(plain, checked):
        assert torch.equal(a, b)
    # the two-call form and the device-count forms pass the validation too
    shape = nova.BlockShape(c["B"], c["N"], c["C"], c["heads"], c["F"], c["Lmax"], sum(c["ks"]))
    y = torch.empty((shape.M, c["C"]), dtype=torch.bfloat16, device=DEV)
    kv_len = torch.tensor(c["kv_lens"], dtype=torch.int32, device=DEV)
    nova.nova_pruned_block_forward(ctx, nova.BlockWeights(c["wt"], 1e-6), shape, c["x"], keep_idx, cu,
                                   c["k_cache"].clone(), c["v_cache"].clone(), kv_len, True, y)
    x_out = torch.empty_like(c["x"])
    nova.nova_restore_from_cache(ctx, c["x"], y, keep_idx, prune_idx, cu, c["cache_prev"], c["h"], c["w"], x_out, None)
    assert torch.equal(x_out, plain[0])
    big_keep = torch.zeros(c["B"] * c["N"], dtype=torch.int32, device=DEV)
    big_prune = torch.zeros(c["B"] * c["N"], dtype=torch.int32, device=DEV)
    big_keep[: keep_idx.numel()] = keep_idx
    big_prune[: prune_idx.numel()] = prune_idx
    y2 = torch.empty((c["B"] * c["N"], c["C"]), dtype=torch.bfloat16, device=DEV)
    y2[: shape.M] = y
    x_out2 = torch.empty_like(c["x"])
    nova.nova_restore_from_cache_device(ctx, c["x"], y2, big_keep, big_prune, cu, c["cache_prev"], c["h"], c["w"],
                                        x_out2, None)
    assert torch.equal(x_out2, plain[0])
    assert ctx.device_status() == 0


@pytest.mark.parametrize("what", ["keep_too_large", "keep_negative", "keep_not_ascending", "cu_decreasing",
                                  "cu_segment_longer_than_n", "cu_total_differs_from_m", "cu_first_not_zero",
                                  "prune_too_large", "prune_duplicate"])
def test_debug_mode_refuses_corrupt_lists_before_any_use(ctx, what):
    """Each corruption is caught by the validation kernel, which only ever reads the lists
    themselves: the call returns INVALID_ARG, no output row is written, the caches and lengths stay
    as they were, and the context works afterwards."""
    c = _case()
    keep_idx, prune_idx, cu = _lists(ctx, c)
    good = _layer(ctx, c, keep_idx, prune_idx, cu)
    k_bad, p_bad, cu_bad = keep_idx.clone(), prune_idx.clone(), cu.clone()
    N = c["N"]
    if what == "keep_too_large":
        k_bad[149] = N + 100000
    elif what == "keep_negative":
        k_bad[0] = -3
    elif what == "keep_not_ascending":
        k_bad[[10, 11]] = k_bad[[11, 10]]
    elif what == "cu_decreasing":
        cu_bad[1] = 200
        cu_bad[2] = 187 - 40
    elif what == "cu_segment_longer_than_n":
        cu_bad[1] = N + 1
    elif what == "cu_total_differs_from_m":
        cu_bad[3] = 186
    elif what == "cu_first_not_zero":
        cu_bad[0] = 1
    elif what == "prune_too_large":
        p_bad[5] = 1 << 30
    elif what == "prune_duplicate":
        p_bad[7] = p_bad[6]
    ctx.set_debug(True)
    shape = nova.BlockShape(c["B"], N, c["C"], c["heads"], c["F"], c["Lmax"], sum(c["ks"]))
    kc, vc = c["k_cache"].clone(), c["v_cache"].clone()
    kv_len = torch.tensor(c["kv_lens"], dtype=torch.int32, device=DEV)
    x_out = torch.full_like(c["x"], float("nan"))
    cache_out = torch.full_like(c["x"], float("nan"))
    if what.startswith("prune"):
        # the restore step reads the pruned list: refused there too
        y = torch.zeros((shape.M, c["C"]), dtype=torch.bfloat16, device=DEV)
        with pytest.raises(nova.NovaError) as ei:
            nova.nova_restore_from_cache(ctx, c["x"], y, k_bad, p_bad, cu_bad, c["cache_prev"], c["h"], c["w"],
                                         x_out, cache_out)
        assert ei.value.status == 1
    with pytest.raises(nova.NovaError) as ei:
        nova.nova_pruned_layer_forward(ctx, nova.BlockWeights(c["wt"], 1e-6), None, shape, c["x"], k_bad, p_bad,
                                       cu_bad, kc, vc, kv_len, True, c["cache_prev"], c["h"], c["w"], x_out, cache_out)
    assert ei.value.status == 1
    assert "validation" in str(ei.value)
    torch.cuda.synchronize()
    assert torch.isnan(x_out.float()).all() and torch.isnan(cache_out.float()).all()      # nothing was written
    assert torch.equal(kc, c["k_cache"]) and torch.equal(vc, c["v_cache"])
    assert kv_len.cpu().tolist() == c["kv_lens"]
    assert ctx.device_status() == 0
    again = _layer(ctx, c, keep_idx, prune_idx, cu)
    for a, b in zip(good, again):
        assert torch.equal(a, b)


def test_guard_bands_around_every_output(ctx):
    c = _case(seed=9)
    B, N, C, h, w = c["B"], c["N"], c["C"], c["h"], c["w"]
    ks, M = c["ks"], sum(c["ks"])
    V = 1000
    logits = synth.randn_bf16((B, N, V), 3, DEV)
    logits0 = logits.clone()
    ent, mean = Banded((B, N), torch.float32), Banded((B,), torch.float32)
    nova.nova_scale_entropy(ctx, logits, ent.t, mean.t)
    want_ent = oracle.scale_entropy(synth.to_f32_numpy(logits))[0]
    assert np.abs(ent.t.cpu().numpy() - want_ent).max() <= 1e-3
    # selection: lists of exactly the sizes the counts give
    keep_idx, prune_idx = Banded((M,), torch.int32, -7), Banded((B * N - M,), torch.int32, -7)
    cu, pos = Banded((B + 1,), torch.int32, -7), Banded((B, N), torch.int32, -7)
    nova.nova_select_topk(ctx, ent.t, torch.tensor(ks, dtype=torch.int32), keep_idx.t, prune_idx.t, cu.t, pos.t)
    w_keep, w_prune, w_cu, _ = oracle.select_topk(ent.t.cpu().numpy(), ks)
    assert np.array_equal(keep_idx.t.cpu().numpy(), w_keep) and np.array_equal(prune_idx.t.cpu().numpy(), w_prune)
    assert np.array_equal(cu.t.cpu().numpy(), w_cu)
    # block, then restore
    shape = nova.BlockShape(B, N, C, c["heads"], c["F"], c["Lmax"], M)
    ctx.ensure_workspace(shape)
    kc, vc = Banded((B, c["Lmax"], C), torch.bfloat16), Banded((B, c["Lmax"], C), torch.bfloat16)
    kc.t.copy_(c["k_cache"])
    vc.t.copy_(c["v_cache"])
    kv_len = Banded((B,), torch.int32)
    kv_len.t.copy_(torch.tensor(c["kv_lens"], dtype=torch.int32))
    y = Banded((M, C), torch.bfloat16, float("nan"))
    x0 = c["x"].clone()
    bw = nova.BlockWeights(c["wt"], 1e-6)
    nova.nova_pruned_block_forward(ctx, bw, shape, c["x"], keep_idx.t, cu.t, kc.t, vc.t, kv_len.t, True, y.t)
    x_out, cache_out = Banded((B, N, C), torch.bfloat16, float("nan")), Banded((B, N, C), torch.bfloat16, float("nan"))
    nova.nova_restore_from_cache(ctx, c["x"], y.t, keep_idx.t, prune_idx.t, cu.t, c["cache_prev"], h, w,
                                 x_out.t, cache_out.t)
    # the one-call form into its own banded outputs
    kc2, vc2 = Banded((B, c["Lmax"], C), torch.bfloat16), Banded((B, c["Lmax"], C), torch.bfloat16)
    kc2.t.copy_(c["k_cache"])
    vc2.t.copy_(c["v_cache"])
    kv_len2 = Banded((B,), torch.int32)
    kv_len2.t.copy_(torch.tensor(c["kv_lens"], dtype=torch.int32))
    x_out2, cache_out2 = Banded((B, N, C), torch.bfloat16, float("nan")), Banded((B, N, C), torch.bfloat16, float("nan"))
    nova.nova_pruned_layer_forward(ctx, bw, None, shape, c["x"], keep_idx.t, prune_idx.t, cu.t, kc2.t, vc2.t, kv_len2.t,
                                   True, c["cache_prev"], h, w, x_out2.t, cache_out2.t)
    # selection scores
    s_mse, s_mass = Banded((B, N), torch.float32, float("nan")), Banded((B, N), torch.float32, float("nan"))
    nova.nova_score_mse(ctx, c["x"], c["cache_prev"], h, w, s_mse.t)
    nova.nova_score_attention_mass(ctx, c["x"], c["x"], c["k_cache"],
                                   torch.tensor(c["kv_lens"], dtype=torch.int32, device=DEV), c["heads"], s_mass.t)
    assert ctx.device_status() == 0
    torch.cuda.synchronize()
    for name, b in dict(ent=ent, mean=mean, keep_idx=keep_idx, prune_idx=prune_idx, cu=cu, pos=pos, k_cache=kc,
                        v_cache=vc, kv_len=kv_len, y=y, x_out=x_out, cache_out=cache_out, k_cache2=kc2, v_cache2=vc2,
                        kv_len2=kv_len2, x_out2=x_out2, cache_out2=cache_out2, s_mse=s_mse, s_mass=s_mass).items():
        assert b.intact(), f"guard band of {name} was written"
    # inputs came back unchanged; outputs are complete and the two forms agree
    assert torch.equal(logits, logits0) and torch.equal(c["x"], x0)
    assert torch.equal(x_out.t, x_out2.t) and torch.equal(cache_out.t, cache_out2.t)
    assert torch.equal(kc.t, kc2.t) and torch.equal(vc.t, vc2.t) and torch.equal(kv_len.t, kv_len2.t)
    assert torch.isfinite(x_out.t.float()).all() and torch.isfinite(y.t.float()).all()
    assert torch.isfinite(s_mse.t).all() and torch.isfinite(s_mass.t).all()
    # cache rows past each image's new length were not written
    for b in range(B):
        n1 = c["kv_lens"][b] + ks[b]
        assert torch.equal(kc.t[b, n1:], c["k_cache"][b, n1:]) and torch.equal(vc.t[b, n1:], c["v_cache"][b, n1:])


def test_profile_select_brackets_only_the_selected_categories(ctx):
    """nova_profile_select: only launches of the selected kernel categories get event brackets; the
    launch counter counts every launch either way."""
    from paper_2602_01345_b200 import pipeline
    c = _case()
    keep_idx, prune_idx, cu = _lists(ctx, c)
    n0 = pipeline.launch_count(ctx)
    pipeline.profile_begin(ctx, ["attention", "restore"])
    _layer(ctx, c, keep_idx, prune_idx, cu)
    prof = pipeline.profile_end(ctx)
    per_layer = pipeline.launch_count(ctx) - n0
    assert per_layer >= 8                                   # two LayerNorms, four GEMMs, attention, restore
    assert prof["attention"][1] == 1 and prof["restore"][1] == 1 and prof["attention"][0] > 0.0
    assert all(v[1] == 0 for k, v in prof.items() if k not in ("attention", "restore"))
    pipeline.profile_begin(ctx)                             # all categories again
    _layer(ctx, c, keep_idx, prune_idx, cu)
    prof = pipeline.profile_end(ctx)
    assert sum(v[1] for v in prof.values()) == per_layer
    with pytest.raises(AssertionError):
        pipeline.profile_begin(ctx, ["no_such_kernel"])

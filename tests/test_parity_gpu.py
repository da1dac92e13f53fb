"""GPU parity: every C-ABI call against the CPU oracle on the same seeded inputs.

Index outputs, keep counts and cumulative offsets must match bit for bit (the oracle's
selection is run on the entropies the GPU produced, so both decide in the same precision);
entropies within 1e-3 absolute; block outputs within 2e-2 of the output's maximum magnitude
(bf16 operands and bf16 storage between stages against the fp32/fp64 oracle); restored rows
within one bf16 unit in the last place.
"""
import math

import numpy as np
import pytest
import torch

import nova_synth as synth
import oracle
import paper_2602_01345_b200 as nova

pytestmark = pytest.mark.gpu

ENT_TOL = 1e-3
BLOCK_TOL = 2e-2
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = nova.Context(0)
    yield c
    assert c.device_status() == 0
    c.close()


def f32(t):
    return synth.to_f32_numpy(t)


def gpu_entropy(ctx, logits):
    S, N, _ = logits.shape
    ent = torch.empty((S, N), dtype=torch.float32, device=DEV)
    mean = torch.empty((S,), dtype=torch.float32, device=DEV)
    nova.nova_scale_entropy(ctx, logits, ent, mean)
    return ent, mean


def gpu_select(ctx, ent, k, with_pos=True):
    S, N = ent.shape
    k = torch.as_tensor(k, dtype=torch.int32)
    M = int(k.sum())
    keep_idx = torch.full((M,), -7, dtype=torch.int32, device=DEV)
    prune_idx = torch.full((S * N - M,), -7, dtype=torch.int32, device=DEV)
    cu = torch.full((S + 1,), -7, dtype=torch.int32, device=DEV)
    pos = torch.full((S, N), -7, dtype=torch.int32, device=DEV) if with_pos else None
    nova.nova_select_topk(ctx, ent, k, keep_idx, prune_idx, cu, pos)
    return keep_idx, prune_idx, cu, pos


# --------------------------------------------------------------------------- entropy
@pytest.mark.parametrize("S,N,V,dtype", [
    (3, 37, 4096, torch.bfloat16),      # several blocks of 8 rows and a ragged last block
    (2, 16, 4096, torch.float32),
    (1, 9, 1000, torch.bfloat16),       # V below one full register tile
    (2, 5, 8192, torch.bfloat16),       # wider than the register path for bf16 -> streaming kernel
    (1, 3, 24, torch.float32),
])
def test_entropy_matches_oracle(ctx, S, N, V, dtype):
    a = synth.smooth_temperature_field(S, 1, N, seed=3, device=DEV)
    logits = synth.logits_from_temperature(a, V, seed=11, dtype=dtype)
    ent, mean = gpu_entropy(ctx, logits)
    want_ent, want_mean = oracle.scale_entropy(f32(logits))
    assert np.abs(ent.cpu().numpy() - want_ent).max() <= ENT_TOL
    assert np.abs(mean.cpu().numpy() - want_mean).max() <= ENT_TOL
    if V >= 1000 and N >= 9:
        assert want_ent.max() - want_ent.min() > 2.0   # the field really spans low and high entropy


@pytest.mark.parametrize("S,N,V,dtype", [
    (3, 1500, 4096, torch.bfloat16),    # 4500 rows: every ring slot of the persistent kernel is reused
    (2, 700, 2048, torch.bfloat16),     # 4 KiB rows
    (1, 333, 1024, torch.bfloat16),     # 2 KiB rows
    (2, 200, 2048, torch.float32),      # 8 KiB rows of fp32
    (4, 4096, 4096, torch.bfloat16),    # the benchmark's launch: batch 4 at 64 x 64 tokens
])
def test_entropy_persistent_kernel_matches_oracle(ctx, S, N, V, dtype):
    a = synth.smooth_temperature_field(S, 1, N, seed=9, device=DEV)
    logits = synth.logits_from_temperature(a, V, seed=13, dtype=dtype)
    ent, mean = gpu_entropy(ctx, logits)
    want_ent, want_mean = oracle.scale_entropy(f32(logits))
    assert np.abs(ent.cpu().numpy() - want_ent).max() <= ENT_TOL
    assert np.abs(mean.cpu().numpy() - want_mean).max() <= ENT_TOL
    # same launch again: the means come from whichever CTA finishes last, in a fixed order
    ent2, mean2 = gpu_entropy(ctx, logits)
    assert torch.equal(ent, ent2) and torch.equal(mean, mean2)
    assert ctx.device_status() == 0


def test_entropy_persistent_kernel_special_values(ctx):
    V, N = 4096, 300
    z = synth.randn_bf16((1, N, V), 21, DEV, std=2.0)
    z[0, 7, 2048:] = float("-inf")                      # exact path: the finite half only
    z[0, 100] = 0.25                                    # uniform -> ln V
    z[0, 150, 5] = float("nan")
    z[0, 299, 4095] = float("inf")
    ent = torch.empty((1, N), dtype=torch.float32, device=DEV)
    nova.nova_scale_entropy(ctx, z, ent, None)
    e = ent.cpu().numpy()[0]
    zz_ok = np.delete(f32(z), [150, 299], axis=1)
    want, _ = oracle.scale_entropy(zz_ok)
    got = np.delete(e, [150, 299])
    assert np.abs(got - want[0]).max() <= ENT_TOL
    assert abs(e[100] - math.log(V)) <= ENT_TOL
    assert np.isnan(e[150]) and np.isnan(e[299])
    assert ctx.device_status() == 5
    assert ctx.device_status() == 0


def test_entropy_ragged_v_and_row_stride(ctx):
    V, stride = 1003, 1008
    buf = torch.zeros((2, 6, stride), dtype=torch.bfloat16, device=DEV)
    buf[:, :, :V] = synth.randn_bf16((2, 6, V), 5, DEV, std=3.0)
    buf[:, :, V:] = 50.0                                # padding must be ignored
    logits = buf[:, :, :V]
    ent = torch.empty((2, 6), dtype=torch.float32, device=DEV)
    nova.nova_scale_entropy(ctx, logits, ent, None)
    want, _ = oracle.scale_entropy(f32(logits))
    assert np.abs(ent.cpu().numpy() - want).max() <= ENT_TOL


def test_entropy_closed_forms_on_gpu(ctx):
    V = 4096
    z = torch.zeros((1, 4, V), dtype=torch.bfloat16, device=DEV)
    z[0, 0] = 0.5                                       # uniform -> ln V
    z[0, 1, 100] = 100.0                                # one hot -> 0
    z[0, 2, :7] = 3.0                                   # two-level
    z[0, 3, 2048:] = float("-inf")                      # -inf logits contribute nothing -> ln 2048
    ent, _ = gpu_entropy(ctx, z)
    e = ent.cpu().numpy()[0]
    assert abs(e[0] - math.log(V)) <= ENT_TOL
    assert 0.0 <= e[1] < 1e-6                           # exact in the oracle; fp32 rounding of ln s here
    Z = 7 * math.exp(3.0) + (V - 7)
    assert abs(e[2] - (math.log(Z) - 7 * 3.0 * math.exp(3.0) / Z)) <= ENT_TOL
    assert abs(e[3] - math.log(2048)) <= ENT_TOL
    assert ctx.device_status() == 0


def test_entropy_flags_nonfinite(ctx):
    z = synth.randn_bf16((1, 8, 256), 1, DEV)
    z[0, 3, 17] = float("nan")
    z[0, 5, 9] = float("inf")
    ent, _ = gpu_entropy(ctx, z)
    e = ent.cpu().numpy()[0]
    assert np.isnan(e[3]) and np.isnan(e[5]) and np.isfinite(np.delete(e, [3, 5])).all()
    assert ctx.device_status() == 5                     # NOVA_ERR_NONFINITE, then cleared
    assert ctx.device_status() == 0


def test_entropy_empty_and_bad_args(ctx):
    ent = torch.empty((0, 4), dtype=torch.float32, device=DEV)
    nova.nova_scale_entropy(ctx, torch.empty((0, 4, 64), dtype=torch.bfloat16, device=DEV), ent, None)
    base = torch.zeros(4 * 64 + 8, dtype=torch.bfloat16, device=DEV)
    mis = base[1:1 + 4 * 64].view(1, 4, 64)             # 2-byte offset: not 16-byte aligned
    with pytest.raises(nova.NovaError) as ei:
        nova.nova_scale_entropy(ctx, mis, torch.empty((1, 4), dtype=torch.float32, device=DEV), None)
    assert ei.value.status == 3


@pytest.mark.parametrize("L,S,N,V", [
    (3, 2, 700, 4096),      # the persistent kernel over three layers' rows: one launch
    (5, 4, 64, 2048),       # fewer rows per layer than CTAs: rows of several layers inside every CTA
    (2, 2, 9, 1000),        # a shape the persistent kernel does not take: layer by layer
])
def test_entropy_all_layers_in_one_call(ctx, L, S, N, V):
    """The entropy maps of all layers of a scale from separate logits tensors: equal, bit for bit,
    to one nova_scale_entropy call per layer, within tolerance of the oracle, in a single launch
    where the persistent kernel applies."""
    from paper_2602_01345_b200 import pipeline
    a = synth.smooth_temperature_field(S, 1, N, seed=3, device=DEV)
    logits = [synth.logits_from_temperature(a * (0.8 + 0.2 * l), V, seed=40 + l) for l in range(L)]
    ent = torch.full((L, S, N), float("nan"), dtype=torch.float32, device=DEV)
    mean = torch.full((L, S), float("nan"), dtype=torch.float32, device=DEV)
    n0 = pipeline.launch_count(ctx)
    nova.nova_scale_entropy_layers(ctx, logits, ent, mean)
    launches = pipeline.launch_count(ctx) - n0
    assert launches == (1 if V in (2048, 4096) else 2 * L)
    for l in range(L):
        e1, m1 = gpu_entropy(ctx, logits[l])
        assert torch.equal(ent[l], e1) and torch.equal(mean[l], m1)
        want_ent, want_mean = oracle.scale_entropy(f32(logits[l]))
        assert np.abs(ent[l].cpu().numpy() - want_ent).max() <= ENT_TOL
        assert np.abs(mean[l].cpu().numpy() - want_mean).max() <= ENT_TOL
    assert ctx.device_status() == 0


# ------------------------------------------------------- entropy fused with the codebook head
def _head_case(ctx, S, N, C, V, seed, bias=True, sample=None):
    x = synth.activations(S, N, C, seed, DEV)
    w = synth.randn_bf16((V, C), seed + 1, DEV, std=3.0 / math.sqrt(C))     # logits of a few units: entropies spread out
    b = synth.randn_bf16((V,), seed + 2, DEV, std=1.0) if bias else None
    ent = torch.full((S, N), float("nan"), dtype=torch.float32, device=DEV)
    mean = torch.full((S,), float("nan"), dtype=torch.float32, device=DEV)
    nova.nova_head_entropy(ctx, x, w, b, ent, mean)
    assert ctx.device_status() == 0
    got = ent.cpu().numpy()
    assert np.isfinite(got).all()
    bb = f32(b) if bias else None
    if sample is None:
        want, want_mean = oracle.head_entropy(f32(x), f32(w), bb)
        assert np.abs(got - want).max() <= ENT_TOL
        assert np.abs(mean.cpu().numpy() - want_mean).max() <= ENT_TOL
        assert want.max() - want.min() > 0.05
    else:
        flat = f32(x).reshape(S * N, C)
        want, _ = oracle.head_entropy(flat[sample][None], f32(w), bb)
        assert np.abs(got.reshape(-1)[sample] - want[0]).max() <= ENT_TOL
        # the means are the fixed-order means of the entropies the kernel wrote
        assert np.abs(mean.cpu().numpy() - got.astype(np.float64).mean(axis=1)).max() <= 1e-4


@pytest.mark.parametrize("S,N,C,V,bias", [
    (2, 300, 256, 4096, True),       # 600 rows: three 256-row blocks, the last one partial
    (1, 77, 128, 992, False),        # fewer rows than one block; V not a multiple of the 256-column tile
    (3, 256, 512, 2048, True),
])
def test_head_entropy_matches_oracle(ctx, S, N, C, V, bias):
    _head_case(ctx, S, N, C, V, seed=31, bias=bias)


def test_head_entropy_full_size_sampled_rows(ctx):
    """Batch 4 at 64 x 64 tokens, width 2048, V = 4096 (the benchmark's launch): sampled rows."""
    rows = np.array([0, 127, 128, 255, 256, 4095, 4096, 8191, 12287, 12288, 16383])
    _head_case(ctx, 4, 4096, 2048, 4096, seed=37, sample=rows)


def test_head_entropy_closed_form_flag_and_bad_args(ctx):
    S, N, C, V = 1, 64, 128, 512
    x = synth.activations(S, N, C, 3, DEV)
    ent = torch.empty((S, N), dtype=torch.float32, device=DEV)
    nova.nova_head_entropy(ctx, x, torch.zeros((V, C), dtype=torch.bfloat16, device=DEV), None, ent)
    assert np.abs(ent.cpu().numpy() - math.log(V)).max() <= ENT_TOL       # zero head -> uniform
    x[0, 5, 7] = float("inf")
    w = synth.randn_bf16((V, C), 4, DEV, std=0.1)
    nova.nova_head_entropy(ctx, x, w, None, ent)
    e = ent.cpu().numpy()[0]
    assert np.isnan(e[5]) and np.isfinite(np.delete(e, 5)).all()
    assert ctx.device_status() == 5
    with pytest.raises(nova.NovaError) as ei:                             # C not a multiple of 64
        nova.nova_head_entropy(ctx, synth.activations(1, 8, 96, 1, DEV),
                               torch.zeros((V, 96), dtype=torch.bfloat16, device=DEV), None,
                               torch.empty((1, 8), dtype=torch.float32, device=DEV))
    assert ei.value.status == 2


# ---------------------------------------------------------------------------- select
@pytest.mark.parametrize("S,N", [(1, 1), (3, 33), (2, 256), (5, 1000), (2, 4096), (2, 16384)])
def test_select_bit_exact(ctx, S, N):
    g = torch.Generator(device="cpu").manual_seed(S * 100003 + N)
    ent = torch.rand((S, N), generator=g) * 8.0
    if N > 1:
        ent[:, ::5] = ent[:, 1:2]                      # many exact ties
    if N > 8:
        ent[0, 3] = -0.0
        ent[0, 7] = 0.0
    ks = [int(x) for x in torch.randint(0, N + 1, (S,), generator=g)]
    ks[0] = N // 2 if N > 1 else 1
    ent_d = ent.to(DEV)
    keep_idx, prune_idx, cu, pos = gpu_select(ctx, ent_d, ks)
    w_keep, w_prune, w_cu, w_pos = oracle.select_topk(ent.numpy(), ks)
    assert np.array_equal(cu.cpu().numpy(), w_cu)
    assert np.array_equal(keep_idx.cpu().numpy(), w_keep)
    assert np.array_equal(prune_idx.cpu().numpy(), w_prune)
    assert np.array_equal(pos.cpu().numpy(), w_pos)


def test_select_edge_counts_and_many_segments(ctx):
    N = 300
    S = 300                                             # more segments than one launch carries
    g = torch.Generator(device="cpu").manual_seed(9)
    ent = torch.randn((S, N), generator=g)
    ks = [0, N, 1, N - 1] + [int(x) for x in torch.randint(0, N + 1, (S - 4,), generator=g)]
    keep_idx, prune_idx, cu, _ = gpu_select(ctx, ent.to(DEV), ks, with_pos=False)
    w_keep, w_prune, w_cu, _ = oracle.select_topk(ent.numpy(), ks)
    assert np.array_equal(cu.cpu().numpy(), w_cu)
    assert np.array_equal(keep_idx.cpu().numpy(), w_keep)
    assert np.array_equal(prune_idx.cpu().numpy(), w_prune)


@pytest.mark.parametrize("G,S,N", [(3, 4, 1000), (32, 4, 4096), (70, 4, 300), (2, 1, 16384)])
@pytest.mark.parametrize("counts_on_device", [False, True])
def test_select_all_layers_in_one_call(ctx, G, S, N, counts_on_device):
    """The selection of G layers x S images in one call: every layer's index lists, cumulative
    counts and positions equal the oracle's for that layer, with host and with device keep counts.
    (32, 4, 4096) is the benchmark's launch; (70, 4, 300) needs more than 256 segments."""
    from paper_2602_01345_b200 import pipeline
    g = torch.Generator(device="cpu").manual_seed(G * 1009 + N)
    ent = torch.rand((G, S, N), generator=g) * 8.0
    ent[:, :, ::7] = ent[:, :, 1:2]                    # exact ties
    k = torch.randint(0, N + 1, (G, S), generator=g).to(torch.int32)
    k[0, 0], k[-1, -1] = N // 2, N
    if S > 1:
        k[0, 1] = 0
    keep_idx = torch.full((G, S * N), -7, dtype=torch.int32, device=DEV)
    prune_idx = torch.full((G, S * N), -7, dtype=torch.int32, device=DEV)
    cu = torch.full((G, S + 1), -7, dtype=torch.int32, device=DEV)
    pos = torch.full((G, S, N), -7, dtype=torch.int32, device=DEV)
    n0 = pipeline.launch_count(ctx)
    nova.nova_select_topk_grouped(ctx, ent.to(DEV), k.to(DEV) if counts_on_device else k, keep_idx, prune_idx, cu, pos)
    launches = pipeline.launch_count(ctx) - n0
    assert launches == (1 if counts_on_device or G * S <= 256 else 2)
    kk, pp, cc, ps = keep_idx.cpu().numpy(), prune_idx.cpu().numpy(), cu.cpu().numpy(), pos.cpu().numpy()
    for l in range(G):
        w_keep, w_prune, w_cu, w_pos = oracle.select_topk(ent[l].numpy(), k[l].numpy())
        M = int(w_cu[-1])
        assert np.array_equal(cc[l], w_cu), l
        assert np.array_equal(kk[l, :M], w_keep) and np.array_equal(pp[l, : S * N - M], w_prune), l
        assert np.array_equal(ps[l], w_pos), l
        assert (kk[l, M:] == -7).all() and (pp[l, S * N - M:] == -7).all()      # nothing written past the lists


def test_select_teacher_forced_on_gpu_entropy(ctx):
    # the selection is decided on the entropies the GPU computed; the oracle ranks those same values
    B, h, w = 2, 16, 16
    a = synth.smooth_temperature_field(B, h, w, seed=0, device=DEV)
    logits = synth.logits_from_temperature(a, synth.V_CODEBOOK, seed=1)
    ent, mean = gpu_entropy(ctx, logits)
    r = nova.nova_keep_ratios(nova.SchedParams(force_act_scale=10, force_keep_ratio=0.5), 10, 1, h * w,
                              mean.cpu().view(B, 1).expand(B, 10).contiguous())
    assert r["keep"].tolist() == [128, 128]
    keep_idx, prune_idx, cu, pos = gpu_select(ctx, ent, r["keep"])
    w_keep, w_prune, w_cu, w_pos = oracle.select_topk(ent.cpu().numpy(), r["keep"].numpy())
    assert np.array_equal(keep_idx.cpu().numpy(), w_keep)
    assert np.array_equal(prune_idx.cpu().numpy(), w_prune)
    assert np.array_equal(cu.cpu().numpy(), w_cu)
    # and the kept tokens are the high-entropy half of the field
    kept_mean = ent.cpu().numpy()[0][w_keep[:128]].mean()
    assert kept_mean > ent.cpu().numpy()[0].mean()


def test_select_bad_args(ctx):
    ent = torch.zeros((1, 8), dtype=torch.float32, device=DEV)
    out = torch.zeros(16, dtype=torch.int32, device=DEV)
    with pytest.raises(nova.NovaError) as ei:
        nova.nova_select_topk(ctx, ent, torch.tensor([9], dtype=torch.int32), out, out, out, None)
    assert ei.value.status == 1
    big = torch.zeros((1, 16385), dtype=torch.float32, device=DEV)
    with pytest.raises(nova.NovaError) as ei:
        nova.nova_select_topk(ctx, big, torch.tensor([5], dtype=torch.int32), out, out, out, None)
    assert ei.value.status == 2


# --------------------------------------------------------------------------- restore
def _bf16_ulp_ok(got, want):
    """|got - want| within one bf16 unit in the last place of the larger magnitude, plus the
    fp32 evaluation error of a four-term weighted sum of O(1) values (about 8 * 2^-24 * 5),
    which dominates only where the interpolated value cancels to nearly zero."""
    mag = np.maximum(np.abs(got), np.abs(want))
    return (np.abs(got - want) <= mag * 2.0 ** -7 + 4e-6).all()


@pytest.mark.parametrize("B,hp,wp,h,w,C,keep_frac", [
    (2, 13, 13, 16, 16, 1024, 0.5),     # config-1 restore
    (3, 5, 7, 9, 11, 64, 0.3),          # ragged everything, rectangular
    (1, 4, 4, 4, 4, 256, 0.0),          # nothing kept, same-size resize
    (2, 3, 3, 8, 8, 128, 1.0),          # everything kept
])
def test_restore_matches_oracle(ctx, B, hp, wp, h, w, C, keep_frac):
    N = h * w
    x = synth.activations(B, N, C, seed=1, device=DEV)
    cache = synth.residual_cache(B, hp, wp, C, seed=2, device=DEV)
    g = torch.Generator(device="cpu").manual_seed(4)
    ent = torch.rand((B, N), generator=g)
    ks = [int(round(keep_frac * N))] * B
    if 0 < keep_frac < 1 and B > 1:
        ks[1] = max(1, ks[1] // 3)
    keep_idx, prune_idx, cu, _ = gpu_select(ctx, ent.to(DEV), ks)
    M = sum(ks)
    y = synth.randn_bf16((M, C), 7, DEV)
    x_out = torch.full_like(x, float("nan"))
    cache_out = torch.full_like(x, float("nan"))
    nova.nova_restore_from_cache(ctx, x, y, keep_idx, prune_idx, cu, cache, h, w, x_out, cache_out)
    wx, wc = oracle.restore_from_cache(f32(x), f32(y), keep_idx.cpu().numpy(), prune_idx.cpu().numpy(),
                                       cu.cpu().numpy(), f32(cache), h, w)
    gx, gc = f32(x_out), f32(cache_out)
    assert np.isfinite(gx).all() and np.isfinite(gc).all()       # every row was written
    kk, cuu = keep_idx.cpu().numpy(), cu.cpu().numpy()
    for b in range(B):
        kept = kk[cuu[b]:cuu[b + 1]]
        assert np.array_equal(gx[b, kept], f32(y)[cuu[b]:cuu[b + 1]])   # kept rows bit-equal y
    assert _bf16_ulp_ok(gx, wx)
    assert _bf16_ulp_ok(gc, wc)
    # no cache output requested
    x_out2 = torch.empty_like(x)
    nova.nova_restore_from_cache(ctx, x, y, keep_idx, prune_idx, cu, cache, h, w, x_out2, None)
    assert torch.equal(x_out2, x_out)


def test_restore_full_size_1024_shape(ctx):
    """The benchmark's restore launch: batch 4, 64 x 64 tokens from a 48 x 48 residual cache, width
    2048, half of the tokens kept; every output row against the oracle."""
    B, hp, wp, h, w, C = 4, 48, 48, 64, 64, 2048
    N = h * w
    x = synth.activations(B, N, C, seed=41, device=DEV)
    cache = synth.residual_cache(B, hp, wp, C, seed=42, device=DEV)
    ent = torch.rand((B, N), generator=torch.Generator(device="cpu").manual_seed(43))
    ks = [2048, 2048, 1999, 2100]
    keep_idx, prune_idx, cu, _ = gpu_select(ctx, ent.to(DEV), ks)
    M = sum(ks)
    y = synth.randn_bf16((M, C), 44, DEV)
    x_out = torch.full_like(x, float("nan"))
    cache_out = torch.full_like(x, float("nan"))
    nova.nova_restore_from_cache(ctx, x, y, keep_idx, prune_idx, cu, cache, h, w, x_out, cache_out)
    wx, wc = oracle.restore_from_cache(f32(x), f32(y), keep_idx.cpu().numpy(), prune_idx.cpu().numpy(),
                                       cu.cpu().numpy(), f32(cache), h, w)
    assert _bf16_ulp_ok(f32(x_out), wx) and _bf16_ulp_ok(f32(cache_out), wc)


# ----------------------------------------------------------------------------- block
def _run_block(ctx, shape, weights, x, keep_idx, cu, k_cache, v_cache, kv_len, append=True):
    ctx.ensure_workspace(shape)
    y = torch.full((shape.M, shape.C), float("nan"), dtype=torch.bfloat16, device=DEV)
    nova.nova_pruned_block_forward(ctx, weights, shape, x, keep_idx, cu, k_cache, v_cache, kv_len, append, y)
    return y


def _rel_err(got, want):
    return float(np.abs(got - want).max() / np.abs(want).max())


def _block_case(ctx, B, N, C, heads, F, Lmax, ks, kv_lens, seed, rows=None):
    wt = synth.block_weights(C, F, seed, DEV)
    x = synth.activations(B, N, C, seed + 1, DEV)
    k_cache, v_cache, _ = synth.kv_cache(B, Lmax, max(kv_lens), C, seed + 2, DEV)
    kv_len = torch.tensor(kv_lens, dtype=torch.int32, device=DEV)
    # rows past each image's own length hold garbage the kernels must never use
    for b, n in enumerate(kv_lens):
        k_cache[b, n:] = float("nan")
        v_cache[b, n:] = float("nan")
    g = torch.Generator(device="cpu").manual_seed(seed)
    ent = torch.rand((B, N), generator=g)
    keep_idx, prune_idx, cu, _ = gpu_select(ctx, ent.to(DEV), ks)
    M = sum(ks)
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, M)
    k0, v0 = k_cache.clone(), v_cache.clone()
    y = _run_block(ctx, shape, nova.BlockWeights(wt, 1e-6), x, keep_idx, cu, k_cache, v_cache, kv_len)
    assert ctx.device_status() == 0
    wts = {n: f32(t) for n, t in wt.items()}
    kc = np.nan_to_num(f32(k0))
    vc = np.nan_to_num(f32(v0))
    wy, wk, wv = oracle.pruned_block_forward(wts, 1e-6, heads, f32(x), keep_idx.cpu().numpy(), cu.cpu().numpy(),
                                             kc, vc, np.array(kv_lens, np.int32), rows=rows)
    gy = f32(y)
    if rows is not None:
        gy = gy[np.asarray(rows)]
    assert np.isfinite(gy).all()
    assert _rel_err(gy, wy) <= BLOCK_TOL
    # appended cache rows and the advanced lengths
    cuu = cu.cpu().numpy()
    gk, gv = f32(k_cache), f32(v_cache)
    for b in range(B):
        n0, kb = kv_lens[b], ks[b]
        if kb == 0:
            continue
        assert _rel_err(gk[b, n0:n0 + kb], wk[cuu[b]:cuu[b + 1]]) <= BLOCK_TOL
        assert _rel_err(gv[b, n0:n0 + kb], wv[cuu[b]:cuu[b + 1]]) <= BLOCK_TOL
        # rows before the append are untouched
        assert torch.equal(k_cache[b, :n0], k0[b, :n0])
    assert kv_len.cpu().tolist() == [a + b for a, b in zip(kv_lens, ks)]
    return _rel_err(gy, wy)


def test_block_config1_shape(ctx):
    # width 1024, 16 heads x 64, MLP 4096, batch 2, 128 of 256 tokens kept, 424 prior tokens
    _block_case(ctx, B=2, N=256, C=1024, heads=16, F=4096, Lmax=680, ks=[128, 128], kv_lens=[424, 424], seed=0)


def test_block_ragged_small_dh64(ctx):
    # kept counts that are not multiples of the 128-row tile, an empty image, ragged key tails
    _block_case(ctx, B=4, N=200, C=128, heads=2, F=256, Lmax=512, ks=[200, 77, 0, 1],
                kv_lens=[0, 130, 17, 300], seed=3)


def test_block_dh128_several_key_tiles(ctx):
    _block_case(ctx, B=2, N=300, C=256, heads=2, F=512, Lmax=1024, ks=[300, 129], kv_lens=[517, 5], seed=5)


def test_block_keep_all_equals_dense(ctx):
    # keep ratio 1: the compacted call is the dense block on every token
    _block_case(ctx, B=1, N=256, C=128, heads=2, F=256, Lmax=512, ks=[256], kv_lens=[100], seed=7)


def test_block_full_size_1024_shape_sampled_rows(ctx):
    """The 1024x1024 large-model shape in the configuration the benchmark times (batch 4, 4096
    tokens per image, about half kept, 6425 prior tokens, width 2048, 16 heads x 128, MLP 8192),
    with ragged keep counts so the last row tile is partial. The appended K/V rows are compared
    for every kept token; the block output on sampled rows (tile corners, the ragged tail)."""
    ks = [2048, 1901, 2048, 2100]
    M = sum(ks)
    rows = [0, 127, 128, 2047, 2048, 2048 + 1900, M - 2100, M - 130, M - 1]
    _block_case(ctx, B=4, N=4096, C=2048, heads=16, F=8192, Lmax=10521, ks=ks, kv_lens=[6425] * 4, seed=11,
                rows=np.array(rows, np.int32))


def test_block_benchmark_configuration_sampled_rows(ctx):
    """Exactly the launch the benchmark times: batch 4, 2048 of 4096 tokens kept per image, 6425 prior
    keys. 512 attention work items on 148 SMs leave a last wave of 68, which is the partly key-split
    case (444 whole items, 68 shared by two CTAs each); sampled rows include the first and last query
    blocks of every image and heads on both sides of the split."""
    ks = [2048] * 4
    rows = [0, 255, 256, 1791, 1792, 2047, 2048, 4095, 4096, 6143, 6144, 6400, 7935, 7936, 8191]
    _block_case(ctx, B=4, N=4096, C=2048, heads=16, F=8192, Lmax=10521, ks=ks, kv_lens=[6425] * 4, seed=19,
                rows=np.array(rows, np.int32))


def test_block_attention_ragged_mid_size(ctx):
    """Thousands of kept rows per image at head size 128, with keep counts and cache lengths that
    leave partial 256-row query blocks, blocks with only one of the two query tiles in use, and
    ragged last key tiles. K/V appends are compared for every row, the block output on sampled
    rows around the tile and block boundaries."""
    ks = [7000, 6013, 6100 + 260]
    M = sum(ks)
    rows = [0, 127, 128, 255, 256, 511, 512, 6999, 7000, 7000 + 6012, 7000 + 6013, 7000 + 6013 + 6143,
            7000 + 6013 + 6144, M - 1]
    _block_case(ctx, B=3, N=8192, C=256, heads=2, F=512, Lmax=9000, ks=ks, kv_lens=[300, 5, 129], seed=17,
                rows=np.array(rows, np.int32))


def test_block_1024_shape_batch1_keep025_sampled_rows(ctx):
    """One image of the 1024x1024 shape at keep ratio 0.25: 1024 kept rows give only 64 attention work
    items for 148 SMs, so every item is shared by two CTAs (one per half of the keys) whose partial
    results are merged by whichever finishes second."""
    rows = [0, 127, 128, 255, 256, 511, 512, 767, 768, 1023]
    _block_case(ctx, B=1, N=4096, C=2048, heads=16, F=8192, Lmax=10521, ks=[1024], kv_lens=[6425], seed=47,
                rows=np.array(rows, np.int32))


def test_block_output_does_not_depend_on_merge_order(ctx):
    """With every attention work item shared by two CTAs, either CTA of a pair may finish second and
    merge; the block output must be the same bits whichever does. Eight runs of the batch-1,
    keep-0.25 shape (64 items, all shared) give identical outputs."""
    B, N, C, heads, F, Lmax, k, prior = 1, 4096, 2048, 16, 8192, 10521, 1024, 6425
    wt = nova.BlockWeights(synth.block_weights(C, F, 47, DEV), 1e-6)
    x = synth.activations(B, N, C, 48, DEV)
    k_cache, v_cache, _ = synth.kv_cache(B, Lmax, prior, C, 49, DEV)
    ent = torch.rand((B, N), generator=torch.Generator(device="cpu").manual_seed(47))
    keep_idx, _, cu, _ = gpu_select(ctx, ent.to(DEV), [k])
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, k)
    first = None
    for _ in range(8):
        kv_len = torch.tensor([prior], dtype=torch.int32, device=DEV)
        y = _run_block(ctx, shape, wt, x, keep_idx, cu, k_cache, v_cache, kv_len)
        if first is None:
            first = y.clone()
        assert torch.equal(y, first)
    assert ctx.device_status() == 0


@pytest.mark.parametrize("kv_len", [517, 5])
def test_block_key_split_small_cases(ctx, kv_len):
    """Four attention work items on 148 SMs, so each is shared by two CTAs, one per half of the keys.
    The second query block has 44 rows (only one of its two query tiles in use). With 517 prior keys
    there are 7 key tiles (4 + 3, the last one ragged); with 5 there are only 3, too few to share, and
    the first CTA of each pair does all the work."""
    _block_case(ctx, B=1, N=600, C=256, heads=2, F=2048, Lmax=1024, ks=[300], kv_lens=[kv_len], seed=53)


def test_block_512_shape_sampled_rows(ctx):
    """VAR-d30-shaped 512x512 block: width 1920, 30 heads x 64, MLP 7680, last scale 32x32 over 1216
    prior tokens, batch 4, ragged keep counts. Widths that are not multiples of 256 (partial GEMM
    tiles), head size 64, and a mix of the CTA-pair and single-CTA GEMM kernels."""
    ks = [512, 300, 1024, 77]
    M = sum(ks)
    rows = [0, 255, 256, 511, 512, 811, 812, 1835, 1836, M - 1]
    _block_case(ctx, B=4, N=1024, C=1920, heads=30, F=7680, Lmax=2240, ks=ks, kv_lens=[1216] * 4, seed=23,
                rows=np.array(rows, np.int32))


def test_block_2048_shape_sampled_rows(ctx):
    """2048x2048 stress shape: one image, 16384 tokens of which 3277 kept (keep ratio 0.2), attending
    to 26137 prior tokens; width 2048, 16 heads x 128, MLP 8192."""
    k = 16384 - int(0.8 * 16384)
    assert k == 3277
    rows = [0, 127, 128, 255, 256, 3071, 3072, 3199, 3200, k - 1]
    _block_case(ctx, B=1, N=16384, C=2048, heads=16, F=8192, Lmax=42521, ks=[k], kv_lens=[26137], seed=29,
                rows=np.array(rows, np.int32))


def _modulation(B, C, seed, names=nova.MODULATION_NAMES):
    g = torch.Generator(device="cpu").manual_seed(seed)
    return {n: (0.5 * torch.randn((B, C), generator=g)).to(torch.bfloat16).to(DEV) for n in names}


@pytest.mark.parametrize("case", ["small_dh64_ragged", "var_d16_256_shape", "gates_only", "device_count"])
def test_block_adaptive_layernorm_matches_oracle(ctx, case):
    """The block with per-image adaptive-LayerNorm modulation (scale and shift after each LayerNorm,
    a gate on each branch) against the oracle: a small ragged case, the 256x256 VAR-d16 shape (last
    scale, batch 4, half kept, sampled rows), a subset of the terms, and the launch sized by an upper
    bound with the kept count read on the device."""
    if case == "var_d16_256_shape":
        ms = synth.CONFIGS["c2_var_d16_256"]
        B, N, C, heads, F, Lmax = 4, ms.scales[-1] ** 2, ms.C, ms.heads, ms.F, ms.total_tokens
        ks, kv_lens = [128, 97, 128, 160], [Lmax - N] * 4
        rows = np.array([0, 127, 128, 224, 225, 352, 353, sum(ks) - 1], np.int32)
    else:
        B, N, C, heads, F, Lmax = 3, 200, 128, 2, 256, 512
        ks, kv_lens, rows = [200, 77, 1], [0, 130, 300], None
    names = ("gate1", "gate2") if case == "gates_only" else nova.MODULATION_NAMES
    md = _modulation(B, C, 77, names)
    wt = synth.block_weights(C, F, 31, DEV)
    x = synth.activations(B, N, C, 32, DEV)
    k_cache, v_cache, _ = synth.kv_cache(B, Lmax, max(kv_lens), C, 33, DEV)
    kv_len = torch.tensor(kv_lens, dtype=torch.int32, device=DEV)
    ent = torch.rand((B, N), generator=torch.Generator(device="cpu").manual_seed(31))
    keep_idx, _, cu, _ = gpu_select(ctx, ent.to(DEV), ks)
    M = sum(ks)
    on_device = case == "device_count"
    cap = B * N if on_device else M
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, cap)
    ctx.ensure_workspace(shape)
    y = torch.full((cap, C), float("nan"), dtype=torch.bfloat16, device=DEV)
    k0, v0 = k_cache.clone(), v_cache.clone()
    idx_buf = torch.zeros(cap, dtype=torch.int32, device=DEV)
    idx_buf[:M] = keep_idx
    nova.nova_pruned_block_forward_adaln(ctx, nova.BlockWeights(wt, 1e-6), md, shape, x, idx_buf, cu, k_cache, v_cache,
                                         kv_len, True, y, m_on_device=on_device)
    assert ctx.device_status() == 0
    wy, wk, wv = oracle.pruned_block_forward({n: f32(t) for n, t in wt.items()}, 1e-6, heads, f32(x),
                                             keep_idx.cpu().numpy(), cu.cpu().numpy(), f32(k0), f32(v0),
                                             np.array(kv_lens, np.int32), rows=rows,
                                             modulation={n: f32(t) for n, t in md.items()})
    gy = f32(y[:M])
    if rows is not None:
        gy = gy[rows]
    assert np.isfinite(gy).all()
    assert _rel_err(gy, wy) <= BLOCK_TOL
    cuu = cu.cpu().numpy()
    for b in range(B):
        n0, kb = kv_lens[b], ks[b]
        assert _rel_err(f32(k_cache)[b, n0:n0 + kb], wk[cuu[b]:cuu[b + 1]]) <= BLOCK_TOL
        assert _rel_err(f32(v_cache)[b, n0:n0 + kb], wv[cuu[b]:cuu[b + 1]]) <= BLOCK_TOL
    if on_device:
        assert torch.isnan(y[M:].float()).all()          # rows past the device-side count are untouched
    # and the terms really act: the plain block gives something else
    y_plain = _run_block(ctx, nova.BlockShape(B, N, C, heads, F, Lmax, M), nova.BlockWeights(wt, 1e-6), x, keep_idx, cu,
                         k0.clone(), v0.clone(), torch.tensor(kv_lens, dtype=torch.int32, device=DEV))
    assert _rel_err(f32(y_plain)[rows] if rows is not None else f32(y_plain), wy) > 2 * BLOCK_TOL


def test_block_adaptive_layernorm_identity_equals_plain_block(ctx):
    """Zero scale and shift with unit gates, and a NULL modulation, give the plain block bit for bit."""
    B, N, C, heads, F, Lmax = 2, 256, 1024, 16, 4096, 680
    ks, kv_lens = [128, 101], [424, 424]
    wt = nova.BlockWeights(synth.block_weights(C, F, 3, DEV), 1e-6)
    x = synth.activations(B, N, C, 4, DEV)
    k_cache, v_cache, _ = synth.kv_cache(B, Lmax, 424, C, 5, DEV)
    ent = torch.rand((B, N), generator=torch.Generator(device="cpu").manual_seed(3))
    keep_idx, _, cu, _ = gpu_select(ctx, ent.to(DEV), ks)
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, sum(ks))
    kv = lambda: torch.tensor(kv_lens, dtype=torch.int32, device=DEV)
    y_plain = _run_block(ctx, shape, wt, x, keep_idx, cu, k_cache.clone(), v_cache.clone(), kv())
    zeros = torch.zeros((B, C), dtype=torch.bfloat16, device=DEV)
    ones = torch.ones((B, C), dtype=torch.bfloat16, device=DEV)
    ident = dict(shift1=zeros, scale1=zeros, gate1=ones, shift2=zeros, scale2=zeros, gate2=ones)
    for md in (ident, None):
        y = torch.empty_like(y_plain)
        nova.nova_pruned_block_forward_adaln(ctx, wt, md, shape, x, keep_idx, cu, k_cache.clone(), v_cache.clone(),
                                             kv(), True, y)
        assert torch.equal(y, y_plain)
    assert ctx.device_status() == 0


def test_block_without_append_leaves_kv_len(ctx):
    B, N, C, heads, F, Lmax = 1, 64, 128, 2, 256, 256
    wt = synth.block_weights(C, F, 1, DEV)
    x = synth.activations(B, N, C, 2, DEV)
    k_cache, v_cache, kv_len = synth.kv_cache(B, Lmax, 10, C, 3, DEV)
    keep_idx, _, cu, _ = gpu_select(ctx, torch.rand((B, N)).to(DEV), [32])
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, 32)
    _run_block(ctx, shape, nova.BlockWeights(wt), x, keep_idx, cu, k_cache, v_cache, kv_len, append=False)
    assert kv_len.cpu().tolist() == [10]
    assert ctx.device_status() == 0


def test_block_cache_overflow_is_reported_not_written(ctx):
    B, N, C, heads, F, Lmax = 1, 64, 128, 2, 256, 40
    wt = synth.block_weights(C, F, 1, DEV)
    x = synth.activations(B, N, C, 2, DEV)
    k_cache, v_cache, kv_len = synth.kv_cache(B, Lmax, 30, C, 3, DEV)
    k0 = k_cache.clone()
    keep_idx, _, cu, _ = gpu_select(ctx, torch.rand((B, N)).to(DEV), [32])   # 30 + 32 > 40
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, 32)
    _run_block(ctx, shape, nova.BlockWeights(wt), x, keep_idx, cu, k_cache, v_cache, kv_len)
    assert ctx.device_status() == 2                      # NOVA_ERR_SHAPE
    assert torch.equal(k_cache, k0) and kv_len.cpu().tolist() == [30]


def test_block_bad_args(ctx):
    wt = synth.block_weights(128, 256, 1, DEV)
    x = synth.activations(1, 8, 128, 2, DEV)
    k_cache, v_cache, kv_len = synth.kv_cache(1, 16, 0, 128, 3, DEV)
    idx = torch.arange(8, dtype=torch.int32, device=DEV)
    cu = torch.tensor([0, 8], dtype=torch.int32, device=DEV)
    y = torch.empty((8, 128), dtype=torch.bfloat16, device=DEV)
    w = nova.BlockWeights(wt)
    with pytest.raises(nova.NovaError) as ei:            # head dim 32 unsupported
        nova.nova_pruned_block_forward(ctx, w, nova.BlockShape(1, 8, 128, 4, 256, 16, 8), x, idx, cu,
                                       k_cache, v_cache, kv_len, True, y)
    assert ei.value.status == 2
    ctx.set_workspace(torch.empty(256, dtype=torch.uint8, device=DEV))
    with pytest.raises(nova.NovaError) as ei:            # workspace too small
        nova.nova_pruned_block_forward(ctx, w, nova.BlockShape(1, 8, 128, 2, 256, 16, 8), x, idx, cu,
                                       k_cache, v_cache, kv_len, True, y)
    assert ei.value.status == 4


# ------------------------------------------------- block + restore in one call (scattered last epilogue)
@pytest.mark.parametrize("case", ["config1", "ragged_small", "keep_all", "keep_none", "device_count", "modulated",
                                  "no_cache_out", "full_size_1024"])
def test_layer_forward_equals_block_then_restore(ctx, case):
    """nova_pruned_layer_forward (the block's last GEMM scatters the kept rows into x_out and writes
    their residual to cache_out; the restore pass touches pruned rows only) gives bit for bit what
    nova_pruned_block_forward + nova_restore_from_cache give, and both match the oracle's block
    followed by its restore."""
    md = None
    if case == "full_size_1024":
        B, h, w, hp, wp, C, heads, F, Lmax = 4, 64, 64, 48, 48, 2048, 16, 8192, 10521
        ks, kv_lens = [2048, 1901, 2048, 2100], [6425] * 4
    elif case == "config1" or case == "modulated":
        B, h, w, hp, wp, C, heads, F, Lmax = 2, 16, 16, 13, 13, 1024, 16, 4096, 680
        ks, kv_lens = [128, 101], [424, 424]
        if case == "modulated":
            md = _modulation(B, C, 77)
    else:
        B, h, w, hp, wp, C, heads, F, Lmax = 3, 10, 15, 7, 9, 128, 2, 256, 512
        ks = {"keep_all": [150] * 3, "keep_none": [0] * 3}.get(case, [150, 37, 0])
        kv_lens = [0, 130, 17]
    N, M = h * w, sum(ks)
    wt = synth.block_weights(C, F, 31, DEV)
    bw = nova.BlockWeights(wt, 1e-6)
    x = synth.activations(B, N, C, 32, DEV)
    k_cache, v_cache, _ = synth.kv_cache(B, Lmax, max(kv_lens), C, 33, DEV)
    cache_prev = synth.residual_cache(B, hp, wp, C, 34, DEV)
    ent = torch.rand((B, N), generator=torch.Generator(device="cpu").manual_seed(31))
    on_device = case == "device_count"
    cap = B * N if on_device else M
    keep_idx = torch.zeros(max(cap, 1), dtype=torch.int32, device=DEV)
    prune_idx = torch.zeros(B * N, dtype=torch.int32, device=DEV)
    cu = torch.empty(B + 1, dtype=torch.int32, device=DEV)
    nova.nova_select_topk(ctx, ent.to(DEV), torch.tensor(ks, dtype=torch.int32), keep_idx[:M], prune_idx[: B * N - M], cu, None)
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, cap)
    ctx.ensure_workspace(shape)
    want_cache = case != "no_cache_out"
    # two calls
    ka, va, la = k_cache.clone(), v_cache.clone(), torch.tensor(kv_lens, dtype=torch.int32, device=DEV)
    y = torch.full((max(cap, 1), C), float("nan"), dtype=torch.bfloat16, device=DEV)
    xa = torch.full_like(x, float("nan"))
    ca = torch.full_like(x, float("nan")) if want_cache else None
    if M > 0:
        nova.nova_pruned_block_forward_adaln(ctx, bw, md, shape, x, keep_idx[:cap], cu, ka, va, la, True, y[:cap],
                                             m_on_device=on_device)
    if on_device:
        nova.nova_restore_from_cache_device(ctx, x, y, keep_idx, prune_idx, cu, cache_prev, h, w, xa, ca)
    else:
        nova.nova_restore_from_cache(ctx, x, y[:M], keep_idx[:M], prune_idx[: B * N - M], cu, cache_prev, h, w, xa, ca)
    # one call
    kb, vb, lb = k_cache.clone(), v_cache.clone(), torch.tensor(kv_lens, dtype=torch.int32, device=DEV)
    xb = torch.full_like(x, float("nan"))
    cb = torch.full_like(x, float("nan")) if want_cache else None
    nova.nova_pruned_layer_forward(ctx, bw, md, shape, x, keep_idx[:cap], prune_idx if on_device else prune_idx[: B * N - M],
                                   cu, kb, vb, lb, True, cache_prev, h, w, xb, cb, m_on_device=on_device)
    assert ctx.device_status() == 0
    assert torch.equal(xa, xb) and torch.equal(ka, kb) and torch.equal(va, vb) and torch.equal(la, lb)
    if want_cache:
        assert torch.equal(ca, cb)
    assert torch.isfinite(xb.float()).all()
    # against the oracle (sampled kept rows at the full size; every pruned row in any case)
    ki, pi, cuu = keep_idx[:M].cpu().numpy(), prune_idx[: B * N - M].cpu().numpy(), cu.cpu().numpy()
    rows = None
    if case == "full_size_1024":
        rows = np.array([0, 127, 2047, 2048, 2048 + 1900, M - 2100, M - 1], np.int32)
    mod_np = {n: f32(t) for n, t in md.items()} if md else None
    wy, _, _ = oracle.pruned_block_forward({n: f32(t) for n, t in wt.items()}, 1e-6, heads, f32(x), ki, cuu, f32(k_cache),
                                           f32(v_cache), np.array(kv_lens, np.int32), rows=rows, modulation=mod_np)
    gx = f32(xb)
    rr = np.arange(M) if rows is None else rows
    if M > 0:
        img = np.searchsorted(cuu, rr, side="right") - 1
        assert _rel_err(gx[img, ki[rr]], wy) <= BLOCK_TOL
    y_for_restore = f32(y[:M])                      # teacher-forced: the restore step on the GPU's block output
    wx, wc = oracle.restore_from_cache(f32(x), y_for_restore, ki, pi, cuu, f32(cache_prev), h, w)
    assert _bf16_ulp_ok(gx, wx)
    if want_cache:
        assert _bf16_ulp_ok(f32(cb), wc)


# ------------------------------------------------------------------------ whole step
def test_whole_pruned_step_config1(ctx):
    """entropy -> keep ratios -> top-k -> block on kept rows -> restore, config-1 shapes, each
    stage checked against the oracle fed with the GPU's inputs to that stage."""
    B, h, w, C, heads, F, P = 2, 16, 16, 1024, 16, 4096, 424
    N, Lmax = h * w, 680
    a = synth.smooth_temperature_field(B, h, w, seed=0, device=DEV)
    logits = synth.logits_from_temperature(a, synth.V_CODEBOOK, seed=1)
    wt = synth.block_weights(C, F, 0, DEV)
    x = synth.activations(B, N, C, 1, DEV)
    k_cache, v_cache, kv_len = synth.kv_cache(B, Lmax, P, C, 2, DEV)
    cache_prev = synth.residual_cache(B, 13, 13, C, 3, DEV)
    k0, v0 = k_cache.clone(), v_cache.clone()

    ent, mean = gpu_entropy(ctx, logits)
    w_ent, w_mean = oracle.scale_entropy(f32(logits))
    assert np.abs(ent.cpu().numpy() - w_ent).max() <= ENT_TOL

    hbar = mean.cpu().view(B, 1).expand(B, 10).contiguous()
    sp = dict(force_act_scale=10, force_keep_ratio=0.5)
    r = nova.nova_keep_ratios(nova.SchedParams(**sp), 10, 1, N, hbar)
    wr = oracle.keep_ratios(oracle.SchedParams(**sp), 10, 1, N, hbar.numpy())
    assert np.array_equal(r["keep"].numpy(), wr["keep"]) and np.array_equal(r["act_scale"].numpy(), wr["act_scale"])

    keep_idx, prune_idx, cu, _ = gpu_select(ctx, ent, r["keep"])
    w_keep, w_prune, w_cu, _ = oracle.select_topk(ent.cpu().numpy(), wr["keep"])
    assert np.array_equal(keep_idx.cpu().numpy(), w_keep) and np.array_equal(prune_idx.cpu().numpy(), w_prune)
    assert np.array_equal(cu.cpu().numpy(), w_cu)

    M = int(r["keep"].sum())
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, M)
    y = _run_block(ctx, shape, nova.BlockWeights(wt, 1e-6), x, keep_idx, cu, k_cache, v_cache, kv_len)
    wy, _, _ = oracle.pruned_block_forward({n: f32(t) for n, t in wt.items()}, 1e-6, heads, f32(x), w_keep, w_cu,
                                           f32(k0), f32(v0), np.full(B, P, np.int32))
    assert _rel_err(f32(y), wy) <= BLOCK_TOL

    x_out = torch.empty_like(x)
    cache_out = torch.empty_like(x)
    nova.nova_restore_from_cache(ctx, x, y, keep_idx, prune_idx, cu, cache_prev, h, w, x_out, cache_out)
    wx, wc = oracle.restore_from_cache(f32(x), f32(y), w_keep, w_prune, w_cu, f32(cache_prev), h, w)
    assert _bf16_ulp_ok(f32(x_out), wx) and _bf16_ulp_ok(f32(cache_out), wc)
    # free-running end to end (oracle block output instead of the GPU's): still within the block tolerance
    fx, _ = oracle.restore_from_cache(f32(x), wy, w_keep, w_prune, w_cu, f32(cache_prev), h, w)
    assert _rel_err(f32(x_out), fx) <= BLOCK_TOL
    assert ctx.device_status() == 0


def test_pipeline_literal_schedule_256_shape(ctx):
    """VAR-d16-shaped layers through the pipeline runner with the paper's schedule taken literally
    (no overrides): the scale history puts the inflection at scale 7, so scale 9 (13 x 13 tokens) is
    pruned with Ratio_9 = sigmoid(1 / tau) - lambda tanh(g_9), modulated per layer by Eq. 12-13 on the
    means the GPU measured. Keep counts, activation scale and index lists must equal the oracle's on
    the GPU's own entropies; the final activations follow the oracle run layer by layer."""
    from paper_2602_01345_b200 import pipeline
    ms = synth.CONFIGS["c2_var_d16_256"]
    B, L, t = 2, 3, 9
    h = w = ms.scales[t - 1]
    hp = wp = ms.scales[t - 2]
    N, P, Lmax = h * w, ms.prior_tokens(t), ms.total_tokens
    weights = [synth.block_weights(ms.C, ms.F, 40 + j, DEV) for j in range(L)]
    caches = [synth.kv_cache(B, Lmax, P, ms.C, 50 + j, DEV) for j in range(L)]
    k_caches, v_caches = [c[0] for c in caches], [c[1] for c in caches]
    kv_len = torch.full((L, B), P, dtype=torch.int32, device=DEV)
    cache_prev = [synth.residual_cache(B, hp, wp, ms.C, 60 + j, DEV) for j in range(L)]
    a = synth.smooth_temperature_field(B, h, w, seed=5, device=DEV)
    beta = synth.layer_inverse_temperatures(L, 5)
    logits = [synth.logits_from_temperature(a * float(beta[j]), synth.V_CODEBOOK, 70 + j) for j in range(L)]
    x_in = synth.activations(B, N, ms.C, 80, DEV)
    k0 = [k.clone() for k in k_caches]
    v0 = [v.clone() for v in v_caches]
    # mean entropies of scales 1..8 rise by 1 per scale, then flatten: t* = 7, pruning from scale 8
    hist = torch.tensor([[1, 2, 3, 4, 5, 6, 6, 6, 0]], dtype=torch.float32).repeat(B, 1)

    runner = pipeline.PrunedScaleRunner(ctx, weights, ms.heads, B, h, w, Lmax, k_caches, v_caches, kv_len, cache_prev)
    # scale 9's own mean entropy (layer 1's map) completes the history, as the caller would do
    ent0, mean0 = gpu_entropy(ctx, logits[0])
    hist[:, t - 1] = mean0.cpu()
    sched = nova.SchedParams()
    x_out, keeps = runner.run_scale(x_in, logits, sched, t, hist)
    assert ctx.device_status() == 0

    osched = oracle.SchedParams()
    x_ref = f32(x_in)
    hbar_layer = np.zeros((B, L), np.float32)
    for j in range(L):
        ent_gpu = runner.ent[j].cpu().numpy()
        w_ent, _ = oracle.scale_entropy(f32(logits[j]))
        assert np.abs(ent_gpu - w_ent).max() <= ENT_TOL
        hbar_layer[:, j] = runner.mean[j].cpu().numpy()
        wr = oracle.keep_ratios(osched, t, j + 1, N, hist.numpy(), hbar_layer[:, : j + 1].copy())
        assert np.array_equal(keeps[j].numpy(), wr["keep"])
        assert (wr["act_scale"] == 8).all() and (wr["t_star"] == 7).all()
        assert (wr["keep"] < N).all() and (wr["keep"] >= 1).all()          # this scale really is pruned
        w_keep, w_prune, w_cu, _ = oracle.select_topk(ent_gpu, wr["keep"])
        wy, _, _ = oracle.pruned_block_forward({n: f32(v) for n, v in weights[j].items()}, 1e-6, ms.heads, x_ref,
                                               w_keep, w_cu, f32(k0[j]), f32(v0[j]), np.full(B, P, np.int32))
        x_ref, _ = oracle.restore_from_cache(x_ref, wy, w_keep, w_prune, w_cu, f32(cache_prev[j]), h, w)
    assert keeps[1].tolist() != keeps[0].tolist() or keeps[2].tolist() != keeps[0].tolist()   # Eq. 13 moved them
    # free-running over three layers: bf16 storage between stages on the GPU, fp32 in the oracle
    assert _rel_err(f32(x_out), x_ref) <= BLOCK_TOL
    assert kv_len.cpu().tolist() == [[P + int(k) for k in keeps[j].tolist()] for j in range(L)]


def test_multi_scale_generation_256_shape(ctx):
    """All ten scales of the VAR-d16 256x256 schedule (1, 2, 3, 4, 5, 6, 8, 10, 13, 16) through two
    layers for two images, with the paper's hyper-parameters and nothing forced: mean entropies that
    follow a seeded sigmoid per image, so the inflection test of Eq. 8-10 fires at a seed-determined
    scale; from the scale after it tokens are pruned by Eq. 11-13; K/V caches grow scale by scale and
    each scale's residual cache (Eq. 15) fills the next scale's pruned rows (Eq. 16). The oracle runs
    the same generation with its own caches; decisions (inflection scale, keep counts, index lists)
    are taken on the entropies the GPU measured and must agree exactly."""
    from paper_2602_01345_b200 import pipeline
    ms = synth.CONFIGS["c2_var_d16_256"]
    B, L, T = 2, 2, len(ms.scales)
    C, Lmax = ms.C, ms.total_tokens
    weights = [synth.block_weights(C, ms.F, 100 + j, DEV) for j in range(L)]
    wts = [{n: f32(v) for n, v in weights[j].items()} for j in range(L)]
    a_env, _ = synth.scale_envelope_temperatures(B, T, seed=3)
    beta = synth.layer_inverse_temperatures(L, 3)
    gen = pipeline.MultiScaleRunner(ctx, weights, ms.heads, B, ms.scales)
    sched, osched = nova.SchedParams(), oracle.SchedParams()
    # the oracle's own state
    ok_cache = [np.zeros((B, Lmax, C), np.float32) for _ in range(L)]
    ov_cache = [np.zeros((B, Lmax, C), np.float32) for _ in range(L)]
    o_len = np.zeros((L, B), np.int32)
    o_res = [None] * L
    pruned_scales = 0
    for t in range(1, T + 1):
        side = ms.scales[t - 1]
        N = side * side
        x_in = synth.activations(B, N, C, 200 + t, DEV)
        a = a_env[:, t - 1].view(B, 1).expand(B, N).contiguous().to(DEV)
        scale_logits = synth.logits_from_temperature(a, synth.V_CODEBOOK, 300 + t)
        layer_logits = [synth.logits_from_temperature(a * float(beta[j]), synth.V_CODEBOOK, 400 + 10 * t + j)
                        for j in range(L)]
        x_out, keeps, runner = gen.run_scale(t, x_in, scale_logits, layer_logits, sched)
        assert ctx.device_status() == 0
        hist = gen.hbar_scale.numpy()
        _, w_mean = oracle.scale_entropy(f32(scale_logits))
        assert np.abs(hist[:, t - 1] - w_mean).max() <= ENT_TOL
        x_ref = f32(x_in)
        hbar_layer = np.zeros((B, L), np.float32)
        for j in range(L):
            ent_gpu = runner.ent[j].cpu().numpy()
            hbar_layer[:, j] = runner.mean[j].cpu().numpy()
            wr = oracle.keep_ratios(osched, t, j + 1, N, hist.copy(), hbar_layer[:, : j + 1].copy())
            assert np.array_equal(keeps[j].numpy(), wr["keep"]), (t, j)
            w_keep, w_prune, w_cu, _ = oracle.select_topk(ent_gpu, wr["keep"])
            wy, wk, wv = oracle.pruned_block_forward(wts[j], 1e-6, ms.heads, x_ref, w_keep, w_cu,
                                                     ok_cache[j], ov_cache[j], o_len[j].copy())
            for b in range(B):
                kb = int(wr["keep"][b])
                ok_cache[j][b, o_len[j, b]:o_len[j, b] + kb] = wk[w_cu[b]:w_cu[b + 1]]
                ov_cache[j][b, o_len[j, b]:o_len[j, b] + kb] = wv[w_cu[b]:w_cu[b + 1]]
                o_len[j, b] += kb
            prev = o_res[j] if o_res[j] is not None else np.zeros((B, 1, 1, C), np.float32)
            x_ref, o_res_new = oracle.restore_from_cache(x_ref, wy, w_keep, w_prune, w_cu, prev, side, side)
            o_res[j] = o_res_new.reshape(B, side, side, C)
            if (wr["keep"] < N).any():
                pruned_scales += 1 if j == 0 else 0
        assert _rel_err(f32(x_out), x_ref) <= BLOCK_TOL, t
        assert gen.kv_len.cpu().numpy().tolist() == o_len.tolist()
    final = oracle.keep_ratios(osched, T, 1, ms.scales[-1] ** 2, gen.hbar_scale.numpy())
    assert (final["act_scale"] > 0).any() and (final["act_scale"] <= T).any()     # the trigger fired in time
    assert pruned_scales >= 1                                                      # and scales were pruned
    # the caches the GPU carried agree with the oracle's after all scales
    for j in range(L):
        assert _rel_err(f32(gen.k_caches[j]), ok_cache[j]) <= BLOCK_TOL
        assert _rel_err(f32(gen.res_cache[j]), o_res[j]) <= BLOCK_TOL


def test_keep_ratios_device_against_oracle(ctx):
    """Eq. 8-13 evaluated by one device thread per image: inflection scale, activation scale and keep
    counts equal the oracle's on seeded sigmoid-shaped entropy histories, at every scale and for
    several layers (layer linkage on random layer means)."""
    B, T, L, N = 64, 10, 6, 4096
    _, hbar = synth.scale_envelope_temperatures(B, T, seed=11)
    hist = hbar.t().contiguous().to(DEV)                      # [T, B]
    rng = np.random.default_rng(5)
    layer = torch.from_numpy((hbar[:, -1:].numpy() * (1 + 0.2 * rng.standard_normal((B, L)))).astype(np.float32))
    layer_dev = layer.t().contiguous().to(DEV)                # [L, B]
    sched, osched = nova.SchedParams(), oracle.SchedParams()
    keep = torch.zeros(B, dtype=torch.int32, device=DEV)
    ts = torch.zeros(B, dtype=torch.int32, device=DEV)
    act = torch.zeros(B, dtype=torch.int32, device=DEV)
    fired = 0
    for t in range(1, T + 1):
        for j in (1, 2, L):
            nova.nova_keep_ratios_device(ctx, sched, t, j, N, hist[:t], layer_dev[:j], keep, ts, act)
            want = oracle.keep_ratios(osched, t, j, N, hbar[:, :t].numpy().copy(), layer[:, :j].numpy().copy())
            assert np.array_equal(ts.cpu().numpy(), want["t_star"]), (t, j)
            assert np.array_equal(act.cpu().numpy(), want["act_scale"]), (t, j)
            assert np.array_equal(keep.cpu().numpy(), want["keep"]), (t, j)
            fired += int((want["keep"] < N).sum())
    assert fired > 0
    assert ctx.device_status() == 0


def test_keep_ratios_all_layers_device_against_oracle(ctx):
    """Eq. 8-13 for all layers of a scale in one launch: row j of the keep counts equals the oracle's
    for layer j + 1 on the means of layers 1..j + 1."""
    B, T, L, N = 16, 10, 16, 4096
    _, hbar = synth.scale_envelope_temperatures(B, T, seed=11)
    hist = hbar.t().contiguous().to(DEV)
    rng = np.random.default_rng(5)
    layer = torch.from_numpy((hbar[:, -1:].numpy() * (1 + 0.2 * rng.standard_normal((B, L)))).astype(np.float32))
    layer_dev = layer.t().contiguous().to(DEV)
    keep = torch.zeros((L, B), dtype=torch.int32, device=DEV)
    ts = torch.zeros(B, dtype=torch.int32, device=DEV)
    act = torch.zeros(B, dtype=torch.int32, device=DEV)
    fired = 0
    for t in (5, 7, 8, 10):
        nova.nova_keep_ratios_layers_device(ctx, nova.SchedParams(), t, N, hist[:t], layer_dev, keep, ts, act)
        got = keep.cpu().numpy()
        for j in range(1, L + 1):
            want = oracle.keep_ratios(oracle.SchedParams(), t, j, N, hbar[:, :t].numpy().copy(), layer[:, :j].numpy().copy())
            assert np.array_equal(got[j - 1], want["keep"]), (t, j)
            fired += int((want["keep"] < N).sum())
        assert np.array_equal(ts.cpu().numpy(), want["t_star"]) and np.array_equal(act.cpu().numpy(), want["act_scale"])
    assert fired > 0


def test_select_topk_device_counts(ctx):
    """Selection with the keep counts in device memory: same lists as the host-count call,
    including counts outside [0, N] (clamped) and the 0 and N corners."""
    S, N = 7, 1000
    ent = torch.from_numpy(np.random.default_rng(2).random((S, N), dtype=np.float32)).to(DEV)
    k = torch.tensor([0, N, 1, 999, 500, -3, N + 5], dtype=torch.int32)
    kc = k.clamp(0, N)
    M = int(kc.sum())
    a_keep = torch.full((S * N,), -7, dtype=torch.int32, device=DEV)
    a_prune = torch.full((S * N,), -7, dtype=torch.int32, device=DEV)
    a_cu = torch.zeros(S + 1, dtype=torch.int32, device=DEV)
    a_pos = torch.zeros((S, N), dtype=torch.int32, device=DEV)
    nova.nova_select_topk_device(ctx, ent, k.to(DEV), a_keep, a_prune, a_cu, a_pos)
    w_keep, w_prune, w_cu, w_pos = oracle.select_topk(ent.cpu().numpy(), kc.numpy())
    assert np.array_equal(a_cu.cpu().numpy(), w_cu)
    assert np.array_equal(a_keep[:M].cpu().numpy(), w_keep)
    assert np.array_equal(a_prune[: S * N - M].cpu().numpy(), w_prune)
    assert np.array_equal(a_pos.cpu().numpy(), w_pos)
    assert (a_keep[M:] == -7).all() and (a_prune[S * N - M:] == -7).all()      # nothing written past the lists


def test_device_driven_generation_equals_host_driven(ctx):
    """The ten-scale generation of the 256x256 schedule with every keep count left on the device
    (no host synchronisation inside a scale, launches sized by the upper bound B*N) gives bit for bit
    what the host-driven call sequence gives: outputs, keep counts, K/V caches, residual caches."""
    from paper_2602_01345_b200 import pipeline
    ms = synth.CONFIGS["c2_var_d16_256"]
    B, L, T = 2, 2, len(ms.scales)
    weights = [synth.block_weights(ms.C, ms.F, 100 + j, DEV) for j in range(L)]
    a_env, _ = synth.scale_envelope_temperatures(B, T, seed=3)
    beta = synth.layer_inverse_temperatures(L, 3)
    host = pipeline.MultiScaleRunner(ctx, weights, ms.heads, B, ms.scales)
    devr = pipeline.MultiScaleRunner(ctx, weights, ms.heads, B, ms.scales, on_device=True)
    sched = nova.SchedParams()
    pruned = 0
    for t in range(1, T + 1):
        N = ms.scales[t - 1] ** 2
        x_in = synth.activations(B, N, ms.C, 200 + t, DEV)
        a = a_env[:, t - 1].view(B, 1).expand(B, N).contiguous().to(DEV)
        scale_logits = synth.logits_from_temperature(a, synth.V_CODEBOOK, 300 + t)
        layer_logits = [synth.logits_from_temperature(a * float(beta[j]), synth.V_CODEBOOK, 400 + 10 * t + j)
                        for j in range(L)]
        xh, keeps_h, _ = host.run_scale(t, x_in, scale_logits, layer_logits, sched)
        xh = xh.clone()
        xd, keeps_d, _ = devr.run_scale(t, x_in, scale_logits, layer_logits, sched)
        assert ctx.device_status() == 0
        assert torch.equal(torch.stack(keeps_h), keeps_d.cpu()), t
        assert torch.equal(xh, xd), t
        pruned += int((torch.stack(keeps_h) < N).sum())
    assert pruned > 0
    assert torch.equal(host.kv_len, devr.kv_len)
    assert torch.equal(host.hbar_scale.t().contiguous(), devr.hist_dev.cpu())
    for j in range(L):
        assert torch.equal(host.k_caches[j], devr.k_caches[j]) and torch.equal(host.v_caches[j], devr.v_caches[j])
        assert torch.equal(host.res_cache[j], devr.res_cache[j])


def test_scale_graph_replay(ctx):
    """A pruned scale recorded once in a CUDA graph and replayed: each replay on fresh inputs gives
    what the eager device-driven launches give, and the keep counts follow the inputs (a different
    entropy history changes them without re-recording)."""
    from paper_2602_01345_b200 import pipeline
    ms = synth.CONFIGS["c2_var_d16_256"]
    B, L, T = 2, 3, len(ms.scales)
    side = ms.scales[-1]
    N, V = side * side, synth.V_CODEBOOK
    weights = [synth.block_weights(ms.C, ms.F, 100 + j, DEV) for j in range(L)]
    Lmax = ms.total_tokens
    prior = Lmax - N
    k_caches = [synth.activations(B, Lmax, ms.C, 50 + j, DEV) for j in range(L)]
    v_caches = [synth.activations(B, Lmax, ms.C, 60 + j, DEV) for j in range(L)]
    cache_prev = [synth.activations(B, ms.scales[-2] ** 2, ms.C, 70 + j, DEV).view(B, ms.scales[-2], ms.scales[-2], ms.C)
                  for j in range(L)]
    kv_len = torch.full((L, B), prior, dtype=torch.int32, device=DEV)
    _, hbar = synth.scale_envelope_temperatures(B, T, seed=3)
    hist = hbar.t().contiguous().to(DEV)
    sched = nova.SchedParams()
    r = pipeline.DeviceScaleRunner(ctx, weights, ms.heads, B, side, side, Lmax, k_caches, v_caches, kv_len,
                                   cache_prev, sched, T, hist, V)

    def load(seed, temp):
        r.x_in.copy_(synth.activations(B, N, ms.C, seed, DEV))
        a = torch.full((B, N), temp, device=DEV)
        r.scale_logits.copy_(synth.logits_from_temperature(a, V, seed + 1))
        for j in range(L):
            r.layer_logits[j].copy_(synth.logits_from_temperature(a * (1 + 0.1 * j), V, seed + 2 + j))

    load(500, 1.0)
    r.capture()
    outs = []
    for seed, temp in ((500, 1.0), (600, 3.0)):
        load(seed, temp)
        kv_len.fill_(prior)
        x_eager = r.enqueue(append_kv=False).clone()
        keep_eager = r.keep.clone()
        x_graph = r.replay().clone()
        assert ctx.device_status() == 0
        assert torch.equal(x_graph, x_eager) and torch.equal(r.keep, keep_eager)
        assert torch.equal(kv_len.cpu(), (prior + r.keep.cpu()).to(torch.int32))        # the recorded pass appends
        outs.append(r.keep.cpu().clone())
    assert (outs[0] < N).any()
    assert not torch.equal(outs[0], outs[1])


def test_runners_with_modulation_agree_and_match_oracle(ctx):
    """The scale runners pass per-image adaptive-LayerNorm modulation through: host-driven and
    device-driven runs of two layers of the 256x256 shape agree, and the first layer's output equals
    the oracle's modulated block followed by its restore."""
    from paper_2602_01345_b200 import pipeline
    ms = synth.CONFIGS["c2_var_d16_256"]
    B, L, T = 2, 2, len(ms.scales)
    side = ms.scales[-1]
    N, V, C, Lmax = side * side, synth.V_CODEBOOK, ms.C, ms.total_tokens
    prior = Lmax - N
    weights = [synth.block_weights(C, ms.F, 100 + j, DEV) for j in range(L)]
    mods = [_modulation(B, C, 900 + j) for j in range(L)]
    hp = ms.scales[-2]
    cache_prev = [synth.residual_cache(B, hp, hp, C, 70 + j, DEV) for j in range(L)]
    x_in = synth.activations(B, N, C, 7, DEV)
    a = synth.smooth_temperature_field(B, side, side, 5, a_lo=0.5, a_hi=6.0, device=DEV)
    logits = [synth.logits_from_temperature(a * (1 + 0.1 * j), V, 20 + j) for j in range(L)]
    sched = nova.SchedParams(force_act_scale=T, force_keep_ratio=0.5)
    hbar = torch.linspace(2.0, 7.0, T).repeat(B, 1).contiguous()

    def caches():
        ks, vs = [], []
        for j in range(L):
            k, v, _ = synth.kv_cache(B, Lmax, prior, C, 50 + 2 * j, DEV)
            ks.append(k)
            vs.append(v)
        return ks, vs, torch.full((L, B), prior, dtype=torch.int32, device=DEV)

    k1, v1, len1 = caches()
    host = pipeline.PrunedScaleRunner(ctx, weights, ms.heads, B, side, side, Lmax, k1, v1, len1, cache_prev,
                                      modulation=mods)
    xh, keeps = host.run_scale(x_in, logits, sched, T, hbar)
    xh = xh.clone()
    k2, v2, len2 = caches()
    devr = pipeline.DeviceScaleRunner(ctx, weights, ms.heads, B, side, side, Lmax, k2, v2, len2, cache_prev, sched, T,
                                      hbar.t().contiguous().to(DEV), V, x_in=x_in, layer_logits=logits,
                                      scale_entropy=False, modulation=mods)
    xd = devr.enqueue()
    assert ctx.device_status() == 0
    # Same keep counts and, for the first layer, the same appended keys bit for bit. The outputs may
    # differ by bf16 rounding: the device-driven launch is sized by the upper bound B*N, which here
    # gives the attention kernel enough scratch to share its 32 work items between CTA pairs, while
    # the host-driven launch (sized by the true 256 rows) runs them unsplit.
    assert torch.equal(torch.stack(keeps), devr.keep.cpu())
    assert torch.equal(k1[0], k2[0])
    assert _rel_err(f32(xd), f32(xh)) <= BLOCK_TOL / 2
    # layer 1 against the oracle (teacher-forced on the GPU's entropies)
    k0, v0, _ = synth.kv_cache(B, Lmax, prior, C, 50, DEV)
    w_keep, w_prune, w_cu, _ = oracle.select_topk(host.ent[0].cpu().numpy(), keeps[0].numpy())
    wy, _, _ = oracle.pruned_block_forward({n: f32(t) for n, t in weights[0].items()}, 1e-6, ms.heads, f32(x_in), w_keep,
                                           w_cu, f32(k0), f32(v0), np.full(B, prior, np.int32),
                                           modulation={n: f32(t) for n, t in mods[0].items()})
    w_x1, _ = oracle.restore_from_cache(f32(x_in), wy, w_keep, w_prune, w_cu, f32(cache_prev[0]), side, side)
    # the runner's layer-1 output is x_buf[0]; layer 2 wrote x_buf[1]
    assert _rel_err(f32(host.x_buf[0]), w_x1) <= BLOCK_TOL


def test_selection_on_one_scale_map_gives_nested_sets(ctx):
    """The other reading of how layers get their entropy map: one map per scale, selected on by every
    layer with that layer's keep count. Kept sets of layers with fewer kept tokens are subsets of
    those with more, index lists equal the oracle's on the same map, and the layers' own logits still
    drive the keep counts through their means (Eq. 12-13)."""
    from paper_2602_01345_b200 import pipeline
    ms = synth.CONFIGS["c2_var_d16_256"]
    B, L, T = 2, 3, len(ms.scales)
    side = ms.scales[-1]
    N, V, C, Lmax = side * side, synth.V_CODEBOOK, ms.C, ms.total_tokens
    prior = Lmax - N
    weights = [synth.block_weights(C, ms.F, 100 + j, DEV) for j in range(L)]
    ks, vs = [], []
    for j in range(L):
        k, v, _ = synth.kv_cache(B, Lmax, prior, C, 50 + 2 * j, DEV)
        ks.append(k)
        vs.append(v)
    kv_len = torch.full((L, B), prior, dtype=torch.int32, device=DEV)
    cache_prev = [synth.residual_cache(B, ms.scales[-2], ms.scales[-2], C, 70 + j, DEV) for j in range(L)]
    x_in = synth.activations(B, N, C, 7, DEV)
    a = synth.smooth_temperature_field(B, side, side, 5, a_lo=0.5, a_hi=6.0, device=DEV)
    beta = [1.0, 0.8, 1.25]
    logits = [synth.logits_from_temperature(a * beta[j], V, 20 + j) for j in range(L)]
    scale_ent = torch.empty((B, N), dtype=torch.float32, device=DEV)
    nova.nova_scale_entropy(ctx, synth.logits_from_temperature(a, V, 19), scale_ent, None)
    _, hbar = synth.scale_envelope_temperatures(B, T, seed=3)
    sched = nova.SchedParams(force_act_scale=T - 1)          # Eq. 11-13 decide the ratios
    runner = pipeline.PrunedScaleRunner(ctx, weights, ms.heads, B, side, side, Lmax, ks, vs, kv_len, cache_prev)
    kept = []
    orig = nova.nova_select_topk

    def spy(ctx_, ent, k, keep_idx, prune_idx, cu_keep, pos=None, stream=None):
        orig(ctx_, ent, k, keep_idx, prune_idx, cu_keep, pos, stream=stream)
        assert ent.data_ptr() == scale_ent.data_ptr()
        w_keep, w_prune, w_cu, _ = oracle.select_topk(scale_ent.cpu().numpy(), k.numpy())
        assert np.array_equal(keep_idx.cpu().numpy(), w_keep) and np.array_equal(cu_keep.cpu().numpy(), w_cu)
        cu = cu_keep.cpu().numpy()
        kept.append([set(keep_idx[cu[b]:cu[b + 1]].cpu().tolist()) for b in range(B)])

    pipeline.nv.nova_select_topk = spy
    try:
        _, keeps = runner.run_scale(x_in, logits, sched, T, hbar.contiguous(), select_ent=scale_ent)
    finally:
        pipeline.nv.nova_select_topk = orig
    assert ctx.device_status() == 0
    counts = torch.stack(keeps)
    assert len({tuple(c.tolist()) for c in counts}) > 1          # the layers' means moved the counts
    for b in range(B):
        order = sorted(range(L), key=lambda j: int(counts[j, b]))
        for lo, hi in zip(order, order[1:]):
            assert kept[lo][b] <= kept[hi][b]


# ------------------------------------------------------------------ alternative selection scores
SCORE_TOL = 2e-3          # relative to the largest score: fp32 sums of products of exact bf16 inputs


@pytest.mark.parametrize("B,hp,wp,h,w,C", [(2, 13, 13, 16, 16, 1024), (3, 5, 7, 9, 11, 64), (1, 4, 4, 4, 4, 256),
                                            (4, 48, 48, 64, 64, 2048)])
def test_score_mse_matches_oracle_and_selects_like_it(ctx, B, hp, wp, h, w, C):
    """The MSE selection score against the oracle on every token, and the selection it drives: the
    oracle's top-k on the GPU's scores equals the GPU's index lists."""
    N = h * w
    ref = synth.residual_cache(B, hp, wp, C, seed=2, device=DEV)
    x = synth.activations(B, N, C, seed=1, device=DEV)
    score = torch.full((B, N), float("nan"), dtype=torch.float32, device=DEV)
    nova.nova_score_mse(ctx, x, ref, h, w, score)
    want = oracle.score_mse(f32(x), f32(ref), h, w)
    got = score.cpu().numpy()
    assert np.abs(got - want).max() <= SCORE_TOL * np.abs(want).max()
    ks = [N // 2] * B
    keep_idx, prune_idx, cu, _ = gpu_select(ctx, score, ks)
    w_keep, w_prune, w_cu, _ = oracle.select_topk(got, ks)
    assert np.array_equal(keep_idx.cpu().numpy(), w_keep) and np.array_equal(prune_idx.cpu().numpy(), w_prune)
    assert ctx.device_status() == 0


@pytest.mark.parametrize("B,N,C,heads,Lmax,kv_lens", [
    (2, 100, 128, 2, 300, [0, 217]),          # head size 64, ragged tiles, one image without prior keys
    (2, 256, 256, 2, 680, [424, 424]),        # head size 128, prior keys of the 256 configuration
    (1, 77, 192, 3, 64, None),                # no cache at all
    (2, 1024, 1920, 30, 2240, [1216, 1216]),  # the 512 configuration's last scale
])
def test_score_attention_mass_matches_oracle(ctx, B, N, C, heads, Lmax, kv_lens):
    """The attention-mass selection score against the oracle on every token (queries scaled up so that
    the rows are peaked and the masses differ by orders of magnitude), reproducible bit for bit, and
    the selection it drives equal to the oracle's on the same scores."""
    q = (synth.activations(B, N, C, 11, DEV).float() * 1.5).to(torch.bfloat16)
    k = synth.activations(B, N, C, 12, DEV)
    if kv_lens is None:
        k_cache = kv_len = None
    else:
        k_cache, _, _ = synth.kv_cache(B, Lmax, max(kv_lens), C, 13, DEV)
        for b, n in enumerate(kv_lens):
            k_cache[b, n:] = float("nan")                 # rows past the length are never read
        kv_len = torch.tensor(kv_lens, dtype=torch.int32, device=DEV)
    score = torch.full((B, N), float("nan"), dtype=torch.float32, device=DEV)
    nova.nova_score_attention_mass(ctx, q, k, k_cache, kv_len, heads, score)
    want = oracle.score_attention_mass(f32(q), f32(k), None if k_cache is None else np.nan_to_num(f32(k_cache)),
                                       None if kv_lens is None else np.array(kv_lens, np.int32), heads)
    got = score.cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= SCORE_TOL * np.abs(want).max()
    assert want.max() - want.min() > 20 * SCORE_TOL * want.max()     # the spread between tokens is far above the tolerance
    if kv_lens is None or min(kv_lens) == 0:
        b0 = 0
        assert abs(float(got[b0].sum()) - 1.0) < 1e-3      # without prior keys all attention stays in the scale
    score2 = torch.empty_like(score)
    nova.nova_score_attention_mass(ctx, q, k, k_cache, kv_len, heads, score2)
    assert torch.equal(score, score2)
    ks = [N // 4] * B
    keep_idx, prune_idx, cu, _ = gpu_select(ctx, score, ks)
    w_keep, w_prune, _, _ = oracle.select_topk(got, ks)
    assert np.array_equal(keep_idx.cpu().numpy(), w_keep) and np.array_equal(prune_idx.cpu().numpy(), w_prune)
    assert ctx.device_status() == 0


def test_score_bad_args(ctx):
    x = synth.activations(1, 16, 64, 1, DEV)
    s = torch.empty((1, 16), dtype=torch.float32, device=DEV)
    with pytest.raises(nova.NovaError) as ei:             # head size 32
        nova.nova_score_attention_mass(ctx, x, x, None, None, 2, s)
    assert ei.value.status == 2
    x2 = synth.activations(1, 16, 60, 1, DEV)
    with pytest.raises(nova.NovaError) as ei:             # C not a multiple of 8
        nova.nova_score_mse(ctx, x2, x2.view(1, 4, 4, 60), 4, 4, s)
    assert ei.value.status == 2


# ------------------------------------------------------------------ bounded device-side waits
def test_device_wait_runs_into_its_limit_and_context_stays_usable():
    """A wait that nothing will ever satisfy (a diagnostic kernel waits on a barrier without a producer)
    ends at the context's wait limit, here 1 ms: the kernel returns, the status word says
    NOVA_ERR_TIMEOUT, and the next ordinary call on the same context is correct. Nothing faults, traps
    or waits without a bound."""
    import time
    c = nova.Context(0)
    try:
        c.set_wait_limit_ns(1_000_000)
        t0 = time.perf_counter()
        c.debug_wait_probe()
        assert c.device_status() == 6                         # NOVA_ERR_TIMEOUT, then cleared
        assert time.perf_counter() - t0 < 0.5                 # milliseconds, not the default second
        assert c.device_status() == 0
        # the limit survives the clearing of the status block: a second probe ends as quickly
        t0 = time.perf_counter()
        c.debug_wait_probe()
        assert c.device_status() == 6 and time.perf_counter() - t0 < 0.5
        # ordinary work on the same context (default limit again), through kernels that wait on barriers themselves
        c.set_wait_limit_ns(0)
        z = synth.randn_bf16((2, 300, 4096), 77, DEV, std=2.0)
        ent, mean = gpu_entropy(c, z)
        want, want_mean = oracle.scale_entropy(f32(z))
        assert np.abs(ent.cpu().numpy() - want).max() <= ENT_TOL
        assert np.abs(mean.cpu().numpy() - want_mean).max() <= ENT_TOL
        _block_case(c, B=1, N=256, C=128, heads=2, F=256, Lmax=512, ks=[200], kv_lens=[100], seed=7)
        assert c.device_status() == 0
    finally:
        c.close()

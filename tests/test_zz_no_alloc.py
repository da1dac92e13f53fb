"""The block entry point for callers that cannot allocate device memory.

Such callers (a plug-in inside a program that owns all device memory and forbids cudaMalloc, a
serving loop that cannot take cudaMalloc's device-wide synchronisation) have no workspace to
give. nova_pruned_block_forward_static takes its scratch from an array inside the library
instead. This test calls it through the C ABI twice in a row, with different shapes so that the
second call meets stale scratch from the first, and checks outputs, appended cache rows and
cache lengths against the ordinary entry point on the same inputs. The file name makes pytest
collect it last.
"""
import numpy as np
import pytest
import torch

import nova_synth as synth
import paper_2602_01345_b200 as nova

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
BLOCK_TOL = 2e-2          # the block tolerance used by the parity tests


def _case(ctx, B, N, C, heads, F, Lmax, ks, kv_lens, seed):
    wt = nova.BlockWeights(synth.block_weights(C, F, seed, DEV), 1e-6)
    x = synth.activations(B, N, C, seed + 1, DEV)
    k_cache, v_cache, _ = synth.kv_cache(B, Lmax, max(kv_lens), C, seed + 2, DEV)
    kv_len = torch.tensor(kv_lens, dtype=torch.int32, device=DEV)
    g = torch.Generator(device="cpu").manual_seed(seed)
    ent = (torch.rand((B, N), generator=g)).to(DEV)
    M = sum(ks)
    keep_idx = torch.empty(M, dtype=torch.int32, device=DEV)
    prune_idx = torch.empty(B * N - M, dtype=torch.int32, device=DEV)
    cu = torch.empty(B + 1, dtype=torch.int32, device=DEV)
    nova.nova_select_topk(ctx, ent, torch.tensor(ks, dtype=torch.int32), keep_idx, prune_idx, cu, None)
    shape = nova.BlockShape(B, N, C, heads, F, Lmax, M)
    return wt, shape, x, keep_idx, cu, k_cache, v_cache, kv_len


def _compare(ctx, case):
    wt, shape, x, keep_idx, cu, k_cache, v_cache, kv_len = case
    # ordinary entry point, with a caller-provided workspace
    ctx.ensure_workspace(shape)
    k_a, v_a, len_a = k_cache.clone(), v_cache.clone(), kv_len.clone()
    y_a = torch.full((shape.M, shape.C), float("nan"), dtype=torch.bfloat16, device=DEV)
    nova.nova_pruned_block_forward(ctx, wt, shape, x, keep_idx, cu, k_a, v_a, len_a, True, y_a)
    # entry point under test: no workspace
    k_b, v_b, len_b = k_cache.clone(), v_cache.clone(), kv_len.clone()
    y_b = torch.full((shape.M, shape.C), float("nan"), dtype=torch.bfloat16, device=DEV)
    nova.nova_pruned_block_forward_static(ctx, wt, shape, x, keep_idx, cu, k_b, v_b, len_b, True, y_b)
    assert ctx.device_status() == 0
    ya, yb = y_a.float().cpu().numpy(), y_b.float().cpu().numpy()
    assert np.isfinite(yb).all()
    assert np.abs(ya - yb).max() <= BLOCK_TOL * np.abs(ya).max()
    for a, b in ((k_a, k_b), (v_a, v_b)):
        fa, fb = a.float().cpu().numpy(), b.float().cpu().numpy()
        assert np.abs(fa - fb).max() <= BLOCK_TOL * np.abs(fa).max()
    assert torch.equal(len_a, len_b)


def test_static_scratch_block_matches_workspace_block_twice():
    ctx = nova.Context(0)
    try:
        assert nova.nova_static_scratch_bytes() >= 4 << 20
        # first call: config-1 shape, the largest that fits (width 1024, MLP 4096, 256 kept rows)
        _compare(ctx, _case(ctx, B=2, N=256, C=1024, heads=16, F=4096, Lmax=680, ks=[128, 128],
                            kv_lens=[424, 424], seed=0))
        # second call straight after: smaller, ragged, head size 128 -> runs over the first call's leftovers
        _compare(ctx, _case(ctx, B=3, N=150, C=256, heads=2, F=512, Lmax=400, ks=[150, 37, 1],
                            kv_lens=[0, 201, 77], seed=4))
        # a shape beyond the built-in array is refused with a clear message, and nothing is launched
        big = nova.BlockShape(4, 4096, 2048, 16, 8192, 10521, 8192)
        assert nova.nova_block_workspace_bytes(big) > nova.nova_static_scratch_bytes()
        dummy = torch.zeros(16, dtype=torch.int32, device=DEV)
        wt = nova.BlockWeights(synth.block_weights(128, 256, 1, DEV))
        with pytest.raises(nova.NovaError) as ei:
            nova.nova_pruned_block_forward_static(ctx, wt, big, dummy, dummy, dummy, dummy, dummy, dummy, True, dummy)
        assert ei.value.status == 4 and "built-in array" in str(ei.value)
    finally:
        ctx.close()

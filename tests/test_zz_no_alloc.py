"""The block entry point for callers that cannot allocate device memory.

Such callers (a plug-in inside a program that owns all device memory and forbids cudaMalloc, a
serving loop that cannot take cudaMalloc's device-wide synchronisation) have no workspace to
give. nova_pruned_block_forward_static takes its scratch from an array inside the library
instead. This test calls it through the C ABI twice in a row, with different shapes so that the
second call meets stale scratch from the first, and checks outputs, appended cache rows and
cache lengths against the ordinary entry point on the same inputs. Both entry points run the
same kernels with the same launch plan, so the comparison is bit for bit (which is inside the
block tolerance of the parity tests, 2e-2 of the output's magnitude). The file name makes
pytest collect it last.
"""
import numpy as np
import pytest
import torch

import nova_synth as synth
import paper_2602_01345_b200 as nova

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


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
    assert np.isfinite(y_b.float().cpu().numpy()).all()
    assert torch.equal(y_a, y_b)
    assert torch.equal(k_a, k_b) and torch.equal(v_a, v_b)
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


def test_static_scratch_block_host_side_returns():
    """Returns decided on the host, before anything is launched: a scale with nothing kept is a no-op
    as for the ordinary entry point, an unsupported shape is refused, and the call is not available
    inside a profiling window or with another device current."""
    from paper_2602_01345_b200 import pipeline
    ctx = nova.Context(0)
    try:
        dummy = torch.zeros(16, dtype=torch.int32, device=DEV)
        wt = nova.BlockWeights(synth.block_weights(128, 256, 1, DEV))
        args = (dummy, dummy, dummy, dummy, dummy, dummy, True, dummy)
        empty = nova.BlockShape(2, 64, 128, 2, 256, 128, 0)            # M == 0: nothing kept
        launches = pipeline.launch_count(ctx)
        nova.nova_pruned_block_forward_static(ctx, wt, empty, *args)
        nova.nova_pruned_block_forward(ctx, wt, empty, *args)
        assert pipeline.launch_count(ctx) == launches
        with pytest.raises(nova.NovaError) as ei:                        # head size 32
            nova.nova_pruned_block_forward_static(ctx, wt, nova.BlockShape(1, 8, 128, 4, 256, 16, 8), *args)
        assert ei.value.status == 2
        ok = nova.BlockShape(1, 8, 128, 2, 256, 16, 8)
        pipeline.profile_begin(ctx)
        try:
            with pytest.raises(nova.NovaError) as ei:
                nova.nova_pruned_block_forward_static(ctx, wt, ok, *args)
            assert ei.value.status == 1 and "profiling" in str(ei.value)
        finally:
            pipeline.profile_end(ctx)
        if torch.cuda.device_count() > 1:
            # the binding makes the context's device current, so go through the raw symbol
            import ctypes as C
            c = ok._c()
            with torch.cuda.device(1):
                st = nova.binding._lib.nova_pruned_block_forward_static(
                    ctx.handle, C.byref(wt.c), C.byref(c), *[dummy.data_ptr()] * 6, 1, dummy.data_ptr(), None)
            assert st == 1
        assert pipeline.launch_count(ctx) == launches
        assert ctx.device_status() == 0
    finally:
        ctx.close()

"""One accelerated scale through all layers: the call sequence a user of the library makes.

The layers' logits are inputs of the scale, so the steps that depend only on them run once for all
layers: entropy maps of every layer (one launch) -> all means to the host in one copy -> keep counts
of every layer from the trigger/ratio functions -> top-k selection of every layer (one launch).
Then for every layer j: block on the kept rows -> restore of the pruned rows from the residual
cache. This module only owns buffers and issues the C-ABI calls in order; it computes nothing itself.
"""
from __future__ import annotations

import ctypes as C

import torch

from . import binding as nv


class PrunedScaleRunner:
    """Buffers and launch sequence for one pruned scale of an L-layer model.

    weights:     list of L dicts of bf16 device tensors (see BlockWeights)
    k_caches / v_caches: lists of L tensors [B, Lmax, C]; kv_len: int32 tensor [L, B]
    cache_prev:  list of L tensors [B, hp, wp, C] (previous scale's residual cache per layer)
    """

    def __init__(self, ctx: nv.Context, weights, n_heads: int, B: int, h: int, w: int, Lmax: int,
                 k_caches, v_caches, kv_len, cache_prev, eps: float = 1e-6, keep_cache_out: bool = True,
                 modulation=None, fused_restore: bool = False):
        """modulation: optional list of L dicts of per-image [B, C] bf16 tensors (adaptive LayerNorm
        of the class-conditional backbones, see nova_pruned_block_forward_adaln).
        fused_restore: run each layer as one nova_pruned_layer_forward call (the block's last GEMM
        scatters the kept rows into x_out / cache_out, the restore pass touches pruned rows only)
        instead of nova_pruned_block_forward + nova_restore_from_cache; same results."""
        self.ctx = ctx
        self.fused_restore = fused_restore
        self.modulation = modulation
        self.L = len(weights)
        self.B, self.h, self.w, self.N = B, h, w, h * w
        self.C = weights[0]["w_o"].shape[0]
        self.F = weights[0]["w_fc1"].shape[0]
        self.n_heads, self.Lmax = n_heads, Lmax
        self.weights = [nv.BlockWeights(wt, eps) for wt in weights]
        self.k_caches, self.v_caches, self.kv_len = k_caches, v_caches, kv_len
        self.cache_prev = cache_prev
        dev = weights[0]["w_o"].device
        self.dev = dev
        N, Cc = self.N, self.C
        self.ent = torch.empty((self.L, B, N), dtype=torch.float32, device=dev)
        self.mean = torch.empty((self.L, B), dtype=torch.float32, device=dev)
        self.mean_host = torch.empty((self.L, B), dtype=torch.float32).pin_memory()
        self.keep_idx = torch.empty((self.L, B * N), dtype=torch.int32, device=dev)      # one list per layer
        self.prune_idx = torch.empty((self.L, B * N), dtype=torch.int32, device=dev)
        self.cu_keep = torch.empty((self.L, B + 1), dtype=torch.int32, device=dev)
        self.y_kept = torch.empty((B * N, Cc), dtype=torch.bfloat16, device=dev)
        self.x_buf = [torch.empty((B, N, Cc), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        self.cache_out = ([torch.empty((B, N, Cc), dtype=torch.bfloat16, device=dev) for _ in range(self.L)]
                          if keep_cache_out else None)
        ctx.ensure_workspace(nv.BlockShape(B, N, Cc, n_heads, self.F, Lmax, B * N))
        self.last_keep = None

    def run_scale(self, x_in, layer_logits, sched: nv.SchedParams, t: int, hbar_scale, append_kv: bool = True,
                  stream=None, logits_ready=None, select_ent=None, layer_hook=None):
        """x_in [B, N, C] bf16; layer_logits: sequence of L tensors [B, N, V]; hbar_scale: CPU
        float32 [B, t] with the mean entropies of scales 1..t. Returns (x_out, keeps) where keeps
        is the list of per-layer keep-count tensors. `logits_ready`, if given, is a list of
        torch.cuda.Event to wait for before layer j's logits are read (upload overlap).
        select_ent: optional device f32 [B, N] entropy map of the scale. If given, every layer selects
        on this one map (the layers' kept sets are then nested: a smaller keep count keeps a subset)
        and the layers' own logits only provide the means of Eq. 12-13; by default layer j selects
        on the entropy map of its own logits.
        layer_hook: optional callable(stage, j, info) called with stage "before" / "after" around layer
        j's launches (info: dict of the tensors involved); for tests that compare layer by layer.
        """
        ctx, B, N = self.ctx, self.B, self.N
        st = stream if stream is not None else torch.cuda.current_stream()
        # The layers' logits are inputs of the scale, not results of its layers, so the entropy maps
        # of a whole group of layers are taken first, in one launch, and their means cross to the host
        # in one copy: one synchronisation per group decides the keep counts of all its layers, and one
        # more launch selects for all of them. With resident logits the group is the whole scale; while
        # logits are still being uploaded a small group lets the blocks of the first layers run under
        # the uploads of the later ones.
        group = self.L if logits_ready is None else min(self.L, 4)
        hbar_layer = torch.zeros((B, self.L), dtype=torch.float32)
        keeps = []
        x = x_in
        for g0 in range(0, self.L, group):
            g1 = min(self.L, g0 + group)
            if logits_ready is not None:
                for j in range(g0, g1):
                    st.wait_event(logits_ready[j])
            nv.nova_scale_entropy_layers(ctx, layer_logits[g0:g1], self.ent[g0:g1], self.mean[g0:g1], stream=st)
            self.mean_host[g0:g1].copy_(self.mean[g0:g1], non_blocking=True)
            st.synchronize()
            hbar_layer[:, g0:g1] = self.mean_host[g0:g1].t()
            keep_all = nv.nova_keep_ratios_layers(sched, t, N, hbar_scale, hbar_layer[:, :g1])["keep"]
            if select_ent is None:
                nv.nova_select_topk_grouped(ctx, self.ent[g0:g1], keep_all[g0:g1], self.keep_idx[g0:g1],
                                            self.prune_idx[g0:g1], self.cu_keep[g0:g1], None, stream=st)
            for j in range(g0, g1):
                keep = keep_all[j]
                M = int(keep.sum())
                keeps.append(keep)
                keep_idx, prune_idx, cu_keep = self.keep_idx[j, :M], self.prune_idx[j, : B * N - M], self.cu_keep[j]
                if select_ent is not None:
                    nv.nova_select_topk(ctx, select_ent, keep, keep_idx, prune_idx, cu_keep, None, stream=st)
                shape = nv.BlockShape(B, N, self.C, self.n_heads, self.F, self.Lmax, M)
                x_out = self.x_buf[j & 1] if x is not self.x_buf[j & 1] else self.x_buf[(j + 1) & 1]
                cache_out = self.cache_out[j] if self.cache_out is not None else None
                if layer_hook is not None:
                    info = dict(x_in=x, x_out=x_out, cache_out=cache_out, keep=keep, keep_idx=keep_idx, prune_idx=prune_idx,
                                cu_keep=cu_keep, k_cache=self.k_caches[j], v_cache=self.v_caches[j], kv_len=self.kv_len[j],
                                cache_prev=self.cache_prev[j], ent=self.ent[j], stream=st)
                    layer_hook("before", j, info)
                if self.fused_restore:
                    nv.nova_pruned_layer_forward(ctx, self.weights[j], self.modulation[j] if self.modulation else None,
                                                 shape, x, keep_idx, prune_idx, cu_keep, self.k_caches[j],
                                                 self.v_caches[j], self.kv_len[j], append_kv, self.cache_prev[j],
                                                 self.h, self.w, x_out, cache_out, stream=st)
                    if layer_hook is not None:
                        layer_hook("after", j, info)
                    x = x_out
                    continue
                if self.modulation is None:
                    nv.nova_pruned_block_forward(ctx, self.weights[j], shape, x, keep_idx, cu_keep,
                                                 self.k_caches[j], self.v_caches[j], self.kv_len[j], append_kv,
                                                 self.y_kept[:M], stream=st)
                else:
                    nv.nova_pruned_block_forward_adaln(ctx, self.weights[j], self.modulation[j], shape, x,
                                                       keep_idx, cu_keep, self.k_caches[j],
                                                       self.v_caches[j], self.kv_len[j], append_kv, self.y_kept[:M],
                                                       stream=st)
                nv.nova_restore_from_cache(ctx, x, self.y_kept[:M], keep_idx, prune_idx,
                                           cu_keep, self.cache_prev[j], self.h, self.w, x_out, cache_out, stream=st)
                if layer_hook is not None:
                    layer_hook("after", j, info)
                x = x_out
        self.last_keep = keeps
        return x, keeps


class MultiScaleRunner:
    """All scales of one generation, in order: the state NOVA carries from scale to scale.

    Per layer it owns the K/V caches (every scale appends the kept tokens' keys and values), the
    residual cache written at the previous scale (Eq. 15; read, resized, at the next one, Eq. 16)
    and, per image, the history of scale mean entropies that the trigger of Eq. 8-10 works on. A
    scale that is not pruned yet is simply the same call sequence with every token kept.
    The backbone around the layers (token embedding, sampling) is not part of this library: the
    caller supplies each scale's layer input and logits.
    """

    def __init__(self, ctx: nv.Context, weights, n_heads: int, B: int, scales, eps: float = 1e-6,
                 on_device: bool = False, fused_restore: bool = False):
        """on_device: keep the entropy history and every keep count in device memory and run each
        scale through DeviceScaleRunner (no host synchronisation inside a scale)."""
        self.ctx, self.weights, self.n_heads, self.B, self.eps = ctx, weights, n_heads, B, eps
        self.on_device = on_device
        self.fused_restore = fused_restore
        self.scales = tuple(scales)
        self.L = len(weights)
        self.C = weights[0]["w_o"].shape[0]
        self.Lmax = sum(s * s for s in self.scales)
        dev = weights[0]["w_o"].device
        self.k_caches = [torch.zeros((B, self.Lmax, self.C), dtype=torch.bfloat16, device=dev) for _ in range(self.L)]
        self.v_caches = [torch.zeros((B, self.Lmax, self.C), dtype=torch.bfloat16, device=dev) for _ in range(self.L)]
        self.kv_len = torch.zeros((self.L, B), dtype=torch.int32, device=dev)
        self.res_cache = [None] * self.L          # previous scale's residual cache per layer, [B, h, w, C]
        self.hbar_scale = torch.zeros((B, 0), dtype=torch.float32)
        self.hist_dev = torch.zeros((len(self.scales), B), dtype=torch.float32, device=dev) if on_device else None
        self.t_done = 0

    def run_scale(self, t: int, x_in, scale_logits, layer_logits, sched: nv.SchedParams, stream=None, layer_hook=None):
        """Scale t (1-based, in order). scale_logits [B, N_t, V] give the scale's mean entropy
        (Eq. 7) that extends the history; layer_logits: L tensors [B, N_t, V]. Returns
        (x_out, keeps, runner) where runner is the PrunedScaleRunner that ran the layers."""
        assert t == self.t_done + 1, "scales must be run in order"
        self.t_done = t
        side = self.scales[t - 1]
        B, N = self.B, side * side
        st = stream if stream is not None else torch.cuda.current_stream()
        if self.on_device:
            runner = DeviceScaleRunner(self.ctx, self.weights, self.n_heads, B, side, side, self.Lmax, self.k_caches,
                                       self.v_caches, self.kv_len, self.res_cache, sched, t, self.hist_dev,
                                       scale_logits.shape[-1], eps=self.eps, logits_dtype=scale_logits.dtype,
                                       fused_restore=self.fused_restore)
            with torch.cuda.stream(st):
                runner.x_in.copy_(x_in)
                runner.scale_logits.copy_(scale_logits)
                for dst, src in zip(runner.layer_logits, layer_logits):
                    dst.copy_(src)
            x_out = runner.enqueue(stream=st)
            self.res_cache = [c.view(B, side, side, self.C) for c in runner.cache_out]
            return x_out, runner.keep, runner
        ent = torch.empty((B, N), dtype=torch.float32, device=x_in.device)
        mean = torch.empty((B,), dtype=torch.float32, device=x_in.device)
        nv.nova_scale_entropy(self.ctx, scale_logits, ent, mean, stream=st)
        self.hbar_scale = torch.cat([self.hbar_scale, mean.cpu().view(B, 1)], dim=1)
        runner = PrunedScaleRunner(self.ctx, self.weights, self.n_heads, B, side, side, self.Lmax, self.k_caches,
                                   self.v_caches, self.kv_len, self.res_cache, eps=self.eps,
                                   fused_restore=self.fused_restore)
        x_out, keeps = runner.run_scale(x_in, layer_logits, sched, t, self.hbar_scale.contiguous(), stream=st,
                                        layer_hook=layer_hook)
        self.res_cache = [c.view(B, side, side, self.C) for c in runner.cache_out]
        return x_out, keeps, runner


class DeviceScaleRunner:
    """One scale through all layers with every decision left on the device.

    For all layers at once: entropy maps and means -> Eq. 8-13 in a one-thread-per-(layer, image)
    kernel -> selection with the keep counts read from device memory. Then per layer the block and
    the restore sized by an upper bound
    (all B*N rows), the kept count read from cu_keep[B]. Nothing crosses to the host, so the whole
    scale is one uninterrupted run of launches that can be recorded in a CUDA graph once and
    replayed for every new batch of the same shape. Inputs live in fixed buffers:
      x_in [B, N, C], scale_logits [B, N, V], layer_logits[j] [B, N, V]   (copy new data in)
      hist [T, B] f32: rows 0..t-2 hold the earlier scales' means; row t-1 is written here.
    Outputs: x_out (property), keep [L, B] int32, cache_out[j] [B, N, C], ent [L, B, N].
    """

    def __init__(self, ctx: nv.Context, weights, n_heads: int, B: int, h: int, w: int, Lmax: int,
                 k_caches, v_caches, kv_len, cache_prev, sched: nv.SchedParams, t: int, hist, V: int,
                 eps: float = 1e-6, logits_dtype=torch.bfloat16, x_in=None, layer_logits=None,
                 scale_entropy: bool = True, modulation=None, fused_restore: bool = False):
        """x_in / layer_logits: existing tensors to use as the fixed input buffers instead of new
        ones. scale_entropy=False: hist row t-1 is already filled by the caller (no scale_logits)."""
        self.ctx, self.sched, self.t = ctx, sched, t
        self.fused_restore = fused_restore    # one nova_pruned_layer_forward call per layer
        self.modulation = modulation          # optional list of L dicts of [B, C] bf16 tensors (fixed buffers)
        self.L = len(weights)
        self.B, self.h, self.w, self.N = B, h, w, h * w
        self.C = weights[0]["w_o"].shape[0]
        self.F = weights[0]["w_fc1"].shape[0]
        self.n_heads, self.Lmax = n_heads, Lmax
        self.weights = [nv.BlockWeights(wt, eps) for wt in weights]
        self.k_caches, self.v_caches, self.kv_len = k_caches, v_caches, kv_len
        dev = weights[0]["w_o"].device
        N, Cc, L = self.N, self.C, self.L
        zero_cache = torch.zeros((B, 1, 1, Cc), dtype=torch.bfloat16, device=dev)
        self.cache_prev = [c if c is not None else zero_cache for c in cache_prev]
        self.hist = hist
        assert hist.dtype == torch.float32 and hist.shape[1] == B and hist.shape[0] >= t and hist.is_contiguous()
        self.x_in = x_in if x_in is not None else torch.empty((B, N, Cc), dtype=torch.bfloat16, device=dev)
        self.scale_logits = torch.empty((B, N, V), dtype=logits_dtype, device=dev) if scale_entropy else None
        self.layer_logits = (list(layer_logits) if layer_logits is not None else
                             [torch.empty((B, N, V), dtype=logits_dtype, device=dev) for _ in range(L)])
        self.ent_scale = torch.empty((B, N), dtype=torch.float32, device=dev)
        self.ent = torch.empty((L, B, N), dtype=torch.float32, device=dev)
        self.mean = torch.empty((L, B), dtype=torch.float32, device=dev)
        self.keep = torch.zeros((L, B), dtype=torch.int32, device=dev)
        self.t_star = torch.zeros((B,), dtype=torch.int32, device=dev)
        self.act_scale = torch.zeros((B,), dtype=torch.int32, device=dev)
        self.keep_idx = torch.empty((L, B * N), dtype=torch.int32, device=dev)       # one list per layer
        self.prune_idx = torch.empty((L, B * N), dtype=torch.int32, device=dev)
        self.cu_keep = torch.zeros((L, B + 1), dtype=torch.int32, device=dev)
        self.y_kept = torch.empty((B * N, Cc), dtype=torch.bfloat16, device=dev)
        self.x_buf = [torch.empty((B, N, Cc), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        self.cache_out = [torch.empty((B, N, Cc), dtype=torch.bfloat16, device=dev) for _ in range(L)]
        self.shape = nv.BlockShape(B, N, Cc, n_heads, self.F, Lmax, B * N)
        ctx.ensure_workspace(self.shape)
        self.x_out = self.x_buf[(L - 1) & 1]
        self.graph = None

    def enqueue(self, append_kv: bool = True, stream=None):
        """Issues the scale's launches on `stream` (default: the current stream); returns x_out."""
        ctx, B, N, t = self.ctx, self.B, self.N, self.t
        st = stream if stream is not None else torch.cuda.current_stream()
        hist_t = self.hist[:t]
        if self.scale_logits is not None:
            nv.nova_scale_entropy(ctx, self.scale_logits, self.ent_scale, hist_t[t - 1], stream=st)
        # everything that depends only on the scale's logits, for all layers at once: three launches
        nv.nova_scale_entropy_layers(ctx, self.layer_logits, self.ent, self.mean, stream=st)
        nv.nova_keep_ratios_layers_device(ctx, self.sched, t, N, hist_t, self.mean, self.keep, self.t_star,
                                          self.act_scale, stream=st)
        nv.nova_select_topk_grouped(ctx, self.ent, self.keep, self.keep_idx, self.prune_idx, self.cu_keep, None,
                                    stream=st)
        x = self.x_in
        for j in range(self.L):
            keep_idx, prune_idx, cu_keep = self.keep_idx[j], self.prune_idx[j], self.cu_keep[j]
            if self.fused_restore:
                x_out = self.x_buf[j & 1]
                nv.nova_pruned_layer_forward(ctx, self.weights[j], self.modulation[j] if self.modulation else None,
                                             self.shape, x, keep_idx, prune_idx, cu_keep, self.k_caches[j],
                                             self.v_caches[j], self.kv_len[j], append_kv, self.cache_prev[j],
                                             self.h, self.w, x_out, self.cache_out[j], m_on_device=True, stream=st)
                x = x_out
                continue
            if self.modulation is None:
                nv.nova_pruned_block_forward_device(ctx, self.weights[j], self.shape, x, keep_idx, cu_keep,
                                                    self.k_caches[j], self.v_caches[j], self.kv_len[j], append_kv,
                                                    self.y_kept, stream=st)
            else:
                nv.nova_pruned_block_forward_adaln(ctx, self.weights[j], self.modulation[j], self.shape, x,
                                                   keep_idx, cu_keep, self.k_caches[j], self.v_caches[j],
                                                   self.kv_len[j], append_kv, self.y_kept, m_on_device=True, stream=st)
            x_out = self.x_buf[j & 1]
            nv.nova_restore_from_cache_device(ctx, x, self.y_kept, keep_idx, prune_idx, cu_keep,
                                              self.cache_prev[j], self.h, self.w, x_out, self.cache_out[j], stream=st)
            x = x_out
        return x

    def capture(self):
        """Records the scale in a CUDA graph. One eager pass without the K/V append comes first (it
        performs the kernels' one-time attribute set-up and leaves kv_len as it was); the recorded
        pass appends."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.enqueue(append_kv=False, stream=side)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.enqueue(append_kv=True)
        self.graph = g
        return g

    def replay(self):
        self.graph.replay()
        return self.x_out


def launch_count(ctx: nv.Context) -> int:
    nv._lib.nova_launch_count.restype = C.c_ulonglong
    nv._lib.nova_launch_count.argtypes = [C.c_void_p]
    return int(nv._lib.nova_launch_count(ctx.handle))


def profile_begin(ctx: nv.Context, categories=None):
    """Starts a profiling window. categories: names of the kernel categories to bracket with events
    (None = all)."""
    lib = nv._lib
    lib.nova_profile_select.argtypes = [C.c_void_p, C.c_ulonglong]
    mask = (1 << 64) - 1
    if categories is not None:
        lib.nova_profile_categories.restype = C.c_int
        lib.nova_profile_category_name.restype = C.c_char_p
        lib.nova_profile_category_name.argtypes = [C.c_int]
        names = [lib.nova_profile_category_name(i).decode() for i in range(lib.nova_profile_categories())]
        unknown = set(categories) - set(names)
        assert not unknown, f"unknown kernel categories {sorted(unknown)}"
        mask = sum(1 << names.index(c) for c in set(categories))
    ctx.check(lib.nova_profile_select(ctx.handle, mask))
    lib.nova_profile_begin.argtypes = [C.c_void_p]
    ctx.check(lib.nova_profile_begin(ctx.handle))


def profile_category_names(ctx: nv.Context) -> list:
    lib = nv._lib
    lib.nova_profile_categories.restype = C.c_int
    lib.nova_profile_category_name.restype = C.c_char_p
    lib.nova_profile_category_name.argtypes = [C.c_int]
    return [lib.nova_profile_category_name(i).decode() for i in range(lib.nova_profile_categories())]


def profile_end(ctx: nv.Context) -> dict:
    """Returns {kernel category: (summed device ms, launches)} for the profiling window."""
    lib = nv._lib
    lib.nova_profile_categories.restype = C.c_int
    lib.nova_profile_category_name.restype = C.c_char_p
    lib.nova_profile_category_name.argtypes = [C.c_int]
    lib.nova_profile_end.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_longlong), C.c_int]
    n = lib.nova_profile_categories()
    ms = (C.c_double * n)()
    cnt = (C.c_longlong * n)()
    ctx.check(lib.nova_profile_end(ctx.handle, ms, cnt, n))
    return {lib.nova_profile_category_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n)}

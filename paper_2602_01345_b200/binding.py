"""ctypes binding of include/nova.h. Names and argument order follow the C ABI."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libnova.so")

STATUS_NAMES = {0: "NOVA_OK", 1: "NOVA_ERR_INVALID_ARG", 2: "NOVA_ERR_SHAPE", 3: "NOVA_ERR_ALIGNMENT",
                4: "NOVA_ERR_WORKSPACE", 5: "NOVA_ERR_NONFINITE", 6: "NOVA_ERR_TIMEOUT", 7: "NOVA_ERR_CUDA"}
NOVA_BF16, NOVA_F32 = 0, 1


class NovaError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


def lib_path() -> str:
    return _LIB_PATH


if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} not found: build it with `python -m paper_2602_01345_b200.build` "
        "(there is no CPU fallback for the NOVA kernels)")


def _stale_sources():
    """Source files newer than the built library (a library built from other sources than the
    ones on disk gives results nobody can account for)."""
    here = os.path.dirname(os.path.abspath(__file__))
    built = os.path.getmtime(_LIB_PATH)
    srcs = [os.path.join(here, "csrc", f) for f in os.listdir(os.path.join(here, "csrc"))]
    srcs.append(os.path.join(os.path.dirname(here), "include", "nova.h"))
    return [p for p in srcs if os.path.exists(p) and os.path.getmtime(p) > built + 1.0]


if _stale_sources() and not os.environ.get("NOVA_ALLOW_STALE_LIBRARY"):
    import warnings
    warnings.warn("libnova.so is older than " + ", ".join(os.path.basename(p) for p in _stale_sources()) +
                  ": rebuild with `python -m paper_2602_01345_b200.build`", RuntimeWarning, stacklevel=2)
_lib = C.CDLL(_LIB_PATH)


class _SchedParams(C.Structure):
    _fields_ = [("t_est", C.c_int), ("alpha", C.c_double), ("tau", C.c_double), ("lam", C.c_double),
                ("k_min", C.c_int), ("ratio_max", C.c_double), ("force_act_scale", C.c_int),
                ("force_keep_ratio", C.c_double)]


_WEIGHT_FIELDS = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
                  "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")


class _BlockWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _WEIGHT_FIELDS] + [("eps", C.c_float)]


class _BlockShape(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("B", "N", "C", "n_heads", "F", "Lmax", "M")]


_vp, _i, _i64 = C.c_void_p, C.c_int, C.c_int64
_lib.nova_create.argtypes = [C.POINTER(_vp), _i]
_lib.nova_create.restype = _i
_lib.nova_destroy.argtypes = [_vp]
_lib.nova_destroy.restype = None
_lib.nova_last_error.argtypes = [_vp]
_lib.nova_last_error.restype = C.c_char_p
_lib.nova_status_string.argtypes = [_i]
_lib.nova_status_string.restype = C.c_char_p
_lib.nova_device_status.argtypes = [_vp, _vp]
_lib.nova_device_status.restype = _i
_lib.nova_set_workspace.argtypes = [_vp, _vp, C.c_size_t]
_lib.nova_set_workspace.restype = _i
_lib.nova_block_workspace_bytes.argtypes = [C.POINTER(_BlockShape)]
_lib.nova_block_workspace_bytes.restype = C.c_size_t
_lib.nova_sched_params_default.argtypes = [C.POINTER(_SchedParams)]
_lib.nova_sched_params_default.restype = None
_lib.nova_scale_entropy.argtypes = [_vp, _vp, _i, _i, _i, _i, _i64, _vp, _vp, _vp]
_lib.nova_scale_entropy.restype = _i
_lib.nova_keep_ratios.argtypes = [C.POINTER(_SchedParams), _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.nova_keep_ratios.restype = _i
_lib.nova_select_topk.argtypes = [_vp, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.nova_select_topk.restype = _i
_lib.nova_pruned_block_forward.argtypes = [_vp, C.POINTER(_BlockWeights), C.POINTER(_BlockShape), _vp, _vp, _vp,
                                           _vp, _vp, _vp, _i, _vp, _vp]
_lib.nova_pruned_block_forward.restype = _i
_lib.nova_restore_from_cache.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp]
_lib.nova_restore_from_cache.restype = _i


def _ptr(t):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the NOVA library must be contiguous"
    return t.data_ptr() if t.numel() > 0 else None


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


@dataclass
class SchedParams:
    """Hyper-parameters of the activation trigger and ratio functions (paper defaults)."""
    t_est: int = 5
    alpha: float = 0.5
    tau: float = 0.8
    lam: float = 0.1
    k_min: int = 1
    ratio_max: float = 1.0
    force_act_scale: int = 0
    force_keep_ratio: float = -1.0

    def _c(self):
        return _SchedParams(self.t_est, self.alpha, self.tau, self.lam, self.k_min, self.ratio_max,
                            self.force_act_scale, self.force_keep_ratio)


@dataclass
class BlockShape:
    B: int
    N: int
    C: int
    n_heads: int
    F: int
    Lmax: int
    M: int

    def _c(self):
        return _BlockShape(self.B, self.N, self.C, self.n_heads, self.F, self.Lmax, self.M)


class BlockWeights:
    """Holds the twelve bf16 device tensors of one block and the C struct that points to them."""

    def __init__(self, tensors: dict, eps: float = 1e-6):
        self.tensors = {n: tensors[n] for n in _WEIGHT_FIELDS}
        for n, t in self.tensors.items():
            assert t.dtype == torch.bfloat16 and t.is_cuda and t.is_contiguous(), n
        self.eps = float(eps)
        self.c = _BlockWeights(*[self.tensors[n].data_ptr() for n in _WEIGHT_FIELDS], self.eps)


class Context:
    """Owns one nova_ctx (one CUDA device) and, optionally, a workspace tensor."""

    def __init__(self, device: int = 0):
        self.device = int(device)
        h = _vp()
        with torch.cuda.device(self.device):
            st = _lib.nova_create(C.byref(h), self.device)
        if st != 0:
            raise NovaError(st, "nova_create failed")
        self.handle = h
        self._workspace = None

    def close(self):
        if getattr(self, "handle", None):
            _lib.nova_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def check(self, status: int):
        if status != 0:
            raise NovaError(status, _lib.nova_last_error(self.handle).decode())

    def set_workspace(self, tensor):
        """Gives the library a device scratch buffer (kept alive by this object)."""
        self._workspace = tensor
        self.check(_lib.nova_set_workspace(self.handle, _ptr(tensor), tensor.numel() * tensor.element_size()
                                           if tensor is not None else 0))

    def ensure_workspace(self, shape: BlockShape):
        need = nova_block_workspace_bytes(shape)
        if self._workspace is None or self._workspace.numel() < need:
            self.set_workspace(torch.empty(need + 256, dtype=torch.uint8, device=f"cuda:{self.device}"))

    def set_wait_limit_ns(self, ns: int):
        """Limit of every device-side wait of this context's later launches (0 = default, 1 s)."""
        _lib.nova_set_wait_limit_ns.argtypes = [_vp, C.c_ulonglong]
        with torch.cuda.device(self.device):
            self.check(_lib.nova_set_wait_limit_ns(self.handle, int(ns)))

    def set_debug(self, on: bool):
        """Debug mode: index lists validated on the device before use, every launch synchronised."""
        _lib.nova_set_debug.argtypes = [_vp, _i]
        _lib.nova_set_debug.restype = _i
        self.check(_lib.nova_set_debug(self.handle, 1 if on else 0))

    def debug_wait_probe(self, stream=None):
        """Launches the diagnostic kernel whose wait can only end by running into the limit."""
        _lib.nova_debug_wait_probe.argtypes = [_vp, _vp]
        self.check(_lib.nova_debug_wait_probe(self.handle, _stream(stream)))

    def device_status(self, stream=None) -> int:
        """Synchronises the stream and returns (and clears) the device status word as a status code."""
        return int(_lib.nova_device_status(self.handle, _stream(stream)))


def nova_block_workspace_bytes(shape: BlockShape) -> int:
    c = shape._c()
    return int(_lib.nova_block_workspace_bytes(C.byref(c)))


def nova_scale_entropy(ctx: Context, logits, ent, mean=None, stream=None):
    """logits [S, N, V] (bf16 or f32, last dim contiguous) -> ent [S, N] f32, mean [S] f32."""
    S, N, V = logits.shape
    assert logits.stride(2) == 1 and logits.stride(0) == N * logits.stride(1)
    dt = {torch.bfloat16: NOVA_BF16, torch.float32: NOVA_F32}[logits.dtype]
    assert ent.dtype == torch.float32 and ent.is_contiguous() and ent.numel() == S * N
    ctx.check(_lib.nova_scale_entropy(ctx.handle, logits.data_ptr() if logits.numel() else None, dt, S, N, V,
                                      logits.stride(1), _ptr(ent), _ptr(mean), _stream(stream)))


_lib.nova_scale_entropy_layers.argtypes = [_vp, C.POINTER(_vp), _i, _i, _i, _i, _i, _i64, _vp, _vp, _vp]
_lib.nova_scale_entropy_layers.restype = _i


def nova_scale_entropy_layers(ctx: Context, layer_logits, ent, mean=None, stream=None):
    """The entropy maps of several layers in one call: layer_logits is a sequence of L tensors
    [S, N, V] (same dtype, shape and row stride) -> ent [L, S, N] f32, mean [L, S] f32."""
    L = len(layer_logits)
    S, N, V = layer_logits[0].shape
    dt = {torch.bfloat16: NOVA_BF16, torch.float32: NOVA_F32}[layer_logits[0].dtype]
    stride = layer_logits[0].stride(1)
    for t in layer_logits:
        assert t.shape == (S, N, V) and t.dtype == layer_logits[0].dtype
        assert t.stride(2) == 1 and t.stride(1) == stride and t.stride(0) == N * stride
    assert ent.dtype == torch.float32 and ent.is_contiguous() and ent.numel() == L * S * N
    assert mean is None or (mean.dtype == torch.float32 and mean.is_contiguous() and mean.numel() == L * S)
    table = (_vp * L)(*[t.data_ptr() if t.numel() else None for t in layer_logits])
    ctx.check(_lib.nova_scale_entropy_layers(ctx.handle, table, L, dt, S, N, V, stride, _ptr(ent), _ptr(mean),
                                             _stream(stream)))


_lib.nova_head_entropy.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp]
_lib.nova_head_entropy.restype = _i


def nova_head_entropy(ctx: Context, x, w_head, b_head, ent, mean=None, stream=None):
    """x [S, N, C] bf16, w_head [V, C] bf16, b_head [V] bf16 or None -> ent [S, N] f32, mean [S] f32:
    entropy of softmax(x @ w_head.T + b_head) per token, logits never stored."""
    S, N, Cc = x.shape
    V = w_head.shape[0]
    assert x.dtype == torch.bfloat16 and x.is_contiguous() and w_head.dtype == torch.bfloat16
    assert w_head.is_contiguous() and w_head.shape[1] == Cc
    assert ent.dtype == torch.float32 and ent.is_contiguous() and ent.numel() == S * N
    ctx.check(_lib.nova_head_entropy(ctx.handle, _ptr(x), _ptr(w_head), _ptr(b_head), S, N, Cc, V,
                                     _ptr(ent), _ptr(mean), _stream(stream)))


def nova_keep_ratios(p: SchedParams, t: int, j: int, N_t: int, hbar_scale, hbar_layer=None):
    """Host arithmetic of the trigger and ratio functions. hbar_* are CPU float32 tensors.

    Returns dict of CPU tensors: t_star, act_scale (int32), ratio_scale, ratio_layer (float64), keep (int32).
    """
    hs = hbar_scale.to("cpu", torch.float32).contiguous()
    B = hs.shape[0]
    assert hs.shape == (B, t)
    hl = None
    if hbar_layer is not None:
        hl = hbar_layer.to("cpu", torch.float32).contiguous()
        assert hl.shape == (B, j)
    out = dict(t_star=torch.zeros(B, dtype=torch.int32), act_scale=torch.zeros(B, dtype=torch.int32),
               ratio_scale=torch.zeros(B, dtype=torch.float64), ratio_layer=torch.zeros(B, dtype=torch.float64),
               keep=torch.zeros(B, dtype=torch.int32))
    c = p._c()
    st = _lib.nova_keep_ratios(C.byref(c), B, t, j, N_t, _ptr(hs), _ptr(hl), _ptr(out["t_star"]),
                               _ptr(out["act_scale"]), _ptr(out["ratio_scale"]), _ptr(out["ratio_layer"]),
                               _ptr(out["keep"]))
    if st != 0:
        raise NovaError(st, "nova_keep_ratios")
    return out


_lib.nova_keep_ratios_layers.argtypes = _lib.nova_keep_ratios.argtypes
_lib.nova_keep_ratios_layers.restype = _i


def nova_keep_ratios_layers(p: SchedParams, t: int, N_t: int, hbar_scale, hbar_layer):
    """Eq. 8-13 for all layers of scale t. hbar_scale CPU f32 [B, t]; hbar_layer CPU f32 [B, L] (the
    means of all L layers). Returns dict: t_star, act_scale int32 [B]; ratio_scale f64 [B];
    ratio_layer f64 [L, B]; keep int32 [L, B]."""
    hs = hbar_scale.to("cpu", torch.float32).contiguous()
    hl = hbar_layer.to("cpu", torch.float32).contiguous()
    B, L = hl.shape
    assert hs.shape == (B, t)
    out = dict(t_star=torch.zeros(B, dtype=torch.int32), act_scale=torch.zeros(B, dtype=torch.int32),
               ratio_scale=torch.zeros(B, dtype=torch.float64), ratio_layer=torch.zeros((L, B), dtype=torch.float64),
               keep=torch.zeros((L, B), dtype=torch.int32))
    c = p._c()
    st = _lib.nova_keep_ratios_layers(C.byref(c), B, t, L, N_t, _ptr(hs), _ptr(hl), _ptr(out["t_star"]),
                                      _ptr(out["act_scale"]), _ptr(out["ratio_scale"]), _ptr(out["ratio_layer"]),
                                      _ptr(out["keep"]))
    if st != 0:
        raise NovaError(st, "nova_keep_ratios_layers")
    return out


_lib.nova_select_topk_grouped.argtypes = [_vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.nova_select_topk_grouped.restype = _i
_lib.nova_select_topk_grouped_device.argtypes = _lib.nova_select_topk_grouped.argtypes
_lib.nova_select_topk_grouped_device.restype = _i


def nova_select_topk_grouped(ctx: Context, ent, k, keep_idx, prune_idx, cu_keep, pos=None, stream=None):
    """Selection for G lists (layers) of S segments each in one launch. ent [G, S, N] f32 device;
    k: int32 [G, S], a CPU tensor (host counts) or a device tensor (counts left on the device);
    keep_idx, prune_idx device int32 [G, S*N]; cu_keep device int32 [G, S+1]; pos [G, S, N] or None."""
    G, S, N = ent.shape
    assert ent.dtype == torch.float32 and ent.is_contiguous()
    assert keep_idx.is_contiguous() and prune_idx.is_contiguous() and cu_keep.is_contiguous()
    assert keep_idx.numel() >= G * S * N and prune_idx.numel() >= G * S * N and cu_keep.numel() >= G * (S + 1)
    if k.is_cuda:
        assert k.dtype == torch.int32 and k.numel() == G * S and k.is_contiguous()
        ctx.check(_lib.nova_select_topk_grouped_device(ctx.handle, _ptr(ent), G, S, N, _ptr(k), _ptr(keep_idx),
                                                       _ptr(prune_idx), _ptr(cu_keep), _ptr(pos), _stream(stream)))
        return
    kk = k.to("cpu", torch.int32).contiguous()
    assert kk.numel() == G * S
    ctx.check(_lib.nova_select_topk_grouped(ctx.handle, _ptr(ent), G, S, N, _ptr(kk), _ptr(keep_idx), _ptr(prune_idx),
                                            _ptr(cu_keep), _ptr(pos), _stream(stream)))


def nova_select_topk(ctx: Context, ent, k, keep_idx, prune_idx, cu_keep, pos=None, stream=None):
    """ent [S, N] f32 device; k: CPU int32 tensor [S]; outputs are device int32 tensors."""
    S, N = ent.shape
    assert ent.dtype == torch.float32 and ent.is_contiguous()
    kk = k.to("cpu", torch.int32).contiguous()
    assert kk.numel() == S
    ctx.check(_lib.nova_select_topk(ctx.handle, _ptr(ent), S, N, _ptr(kk), _ptr(keep_idx), _ptr(prune_idx),
                                    _ptr(cu_keep), _ptr(pos), _stream(stream)))


def nova_pruned_block_forward(ctx: Context, w: BlockWeights, shape: BlockShape, x_in, keep_idx, cu_keep,
                              k_cache, v_cache, kv_len, append_kv, y_kept, stream=None):
    c = shape._c()
    ctx.check(_lib.nova_pruned_block_forward(ctx.handle, C.byref(w.c), C.byref(c), _ptr(x_in), _ptr(keep_idx),
                                             _ptr(cu_keep), _ptr(k_cache), _ptr(v_cache), _ptr(kv_len),
                                             int(bool(append_kv)), _ptr(y_kept), _stream(stream)))


def nova_restore_from_cache(ctx: Context, x_in, y_kept, keep_idx, prune_idx, cu_keep, cache_prev, h, w,
                            x_out, cache_out=None, stream=None):
    B, N, Cc = x_in.shape
    assert N == h * w
    M = int(keep_idx.numel())
    hp, wp = (cache_prev.shape[1], cache_prev.shape[2]) if cache_prev is not None else (0, 0)
    ctx.check(_lib.nova_restore_from_cache(ctx.handle, _ptr(x_in), _ptr(y_kept), _ptr(keep_idx), _ptr(prune_idx),
                                           _ptr(cu_keep), _ptr(cache_prev), hp, wp, h, w, Cc, B, M,
                                           _ptr(x_out), _ptr(cache_out), _stream(stream)))


_lib.nova_static_scratch_bytes.argtypes = []
_lib.nova_static_scratch_bytes.restype = C.c_size_t
_lib.nova_pruned_block_forward_static.argtypes = _lib.nova_pruned_block_forward.argtypes
_lib.nova_pruned_block_forward_static.restype = _i


def nova_static_scratch_bytes() -> int:
    """Size of the scratch array built into the library for nova_pruned_block_forward_static."""
    return int(_lib.nova_static_scratch_bytes())


def nova_pruned_block_forward_static(ctx: Context, w: BlockWeights, shape: BlockShape, x_in, keep_idx, cu_keep,
                                     k_cache, v_cache, kv_len, append_kv, y_kept, stream=None):
    """nova_pruned_block_forward for callers that may not allocate device memory (a plug-in inside
    a host program that owns all device memory, a serving loop that cannot afford cudaMalloc's
    device-wide synchronisation): same arguments and results, but the scratch comes from a fixed
    array inside the library instead of a workspace tensor. Shapes that need more than
    nova_static_scratch_bytes() are refused; calls that overlap on the GPU race on the array.
    """
    c = shape._c()
    with torch.cuda.device(ctx.device):
        ctx.check(_lib.nova_pruned_block_forward_static(
            ctx.handle, C.byref(w.c), C.byref(c), _ptr(x_in), _ptr(keep_idx), _ptr(cu_keep), _ptr(k_cache),
            _ptr(v_cache), _ptr(kv_len), int(bool(append_kv)), _ptr(y_kept), _stream(stream)))


# ---- the device-driven variants: nothing crosses to the host between the calls of a layer -----
_lib.nova_keep_ratios_device.argtypes = [_vp, C.POINTER(_SchedParams), _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.nova_keep_ratios_device.restype = _i
_lib.nova_select_topk_device.argtypes = _lib.nova_select_topk.argtypes
_lib.nova_select_topk_device.restype = _i
_lib.nova_pruned_block_forward_device.argtypes = _lib.nova_pruned_block_forward.argtypes
_lib.nova_pruned_block_forward_device.restype = _i
_lib.nova_restore_from_cache_device.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp]
_lib.nova_restore_from_cache_device.restype = _i


def nova_keep_ratios_device(ctx: Context, p: SchedParams, t: int, j: int, N_t: int, hbar_scale, hbar_layer, keep,
                            t_star=None, act_scale=None, stream=None):
    """Eq. 8-13 on the device. hbar_scale: device f32 [t, B]; hbar_layer: device f32 [j, B] or None;
    keep (and optionally t_star, act_scale): device int32 [B]."""
    B = keep.numel()
    assert hbar_scale.dtype == torch.float32 and hbar_scale.shape == (t, B)
    assert hbar_layer is None or (hbar_layer.dtype == torch.float32 and hbar_layer.shape == (j, B))
    assert keep.dtype == torch.int32
    c = p._c()
    ctx.check(_lib.nova_keep_ratios_device(ctx.handle, C.byref(c), B, t, j, N_t, _ptr(hbar_scale), _ptr(hbar_layer),
                                           _ptr(t_star), _ptr(act_scale), _ptr(keep), _stream(stream)))


_lib.nova_keep_ratios_layers_device.argtypes = _lib.nova_keep_ratios_device.argtypes
_lib.nova_keep_ratios_layers_device.restype = _i


def nova_keep_ratios_layers_device(ctx: Context, p: SchedParams, t: int, N_t: int, hbar_scale, hbar_layer, keep,
                                   t_star=None, act_scale=None, stream=None):
    """Eq. 8-13 for all L layers on the device. hbar_scale device f32 [t, B]; hbar_layer device f32
    [L, B]; keep device int32 [L, B]."""
    L, B = keep.shape
    assert hbar_scale.dtype == torch.float32 and hbar_scale.shape == (t, B)
    assert hbar_layer.dtype == torch.float32 and hbar_layer.shape == (L, B) and hbar_layer.is_contiguous()
    assert keep.dtype == torch.int32 and keep.is_contiguous()
    c = p._c()
    ctx.check(_lib.nova_keep_ratios_layers_device(ctx.handle, C.byref(c), B, t, L, N_t, _ptr(hbar_scale),
                                                  _ptr(hbar_layer), _ptr(t_star), _ptr(act_scale), _ptr(keep),
                                                  _stream(stream)))


def nova_select_topk_device(ctx: Context, ent, k_dev, keep_idx, prune_idx, cu_keep, pos=None, stream=None):
    """nova_select_topk with the keep counts in a device int32 tensor [S]; keep_idx and prune_idx
    must each have room for S*N entries."""
    S, N = ent.shape
    assert ent.dtype == torch.float32 and ent.is_contiguous()
    assert k_dev.dtype == torch.int32 and k_dev.numel() == S and k_dev.is_cuda
    assert keep_idx.numel() >= S * N and prune_idx.numel() >= S * N
    ctx.check(_lib.nova_select_topk_device(ctx.handle, _ptr(ent), S, N, _ptr(k_dev), _ptr(keep_idx), _ptr(prune_idx),
                                           _ptr(cu_keep), _ptr(pos), _stream(stream)))


def nova_pruned_block_forward_device(ctx: Context, w: BlockWeights, shape: BlockShape, x_in, keep_idx, cu_keep,
                                     k_cache, v_cache, kv_len, append_kv, y_kept, stream=None):
    """nova_pruned_block_forward where shape.M is an upper bound; the true count is cu_keep[B]."""
    c = shape._c()
    assert y_kept.shape[0] >= shape.M
    ctx.check(_lib.nova_pruned_block_forward_device(ctx.handle, C.byref(w.c), C.byref(c), _ptr(x_in), _ptr(keep_idx),
                                                    _ptr(cu_keep), _ptr(k_cache), _ptr(v_cache), _ptr(kv_len),
                                                    int(bool(append_kv)), _ptr(y_kept), _stream(stream)))


def nova_restore_from_cache_device(ctx: Context, x_in, y_kept, keep_idx, prune_idx, cu_keep, cache_prev, h, w,
                                   x_out, cache_out=None, stream=None):
    """nova_restore_from_cache with the kept count read from cu_keep[B] on the device."""
    B, N, Cc = x_in.shape
    assert N == h * w and cache_prev is not None
    ctx.check(_lib.nova_restore_from_cache_device(ctx.handle, _ptr(x_in), _ptr(y_kept), _ptr(keep_idx),
                                                  _ptr(prune_idx), _ptr(cu_keep), _ptr(cache_prev),
                                                  cache_prev.shape[1], cache_prev.shape[2], h, w, Cc, B,
                                                  _ptr(x_out), _ptr(cache_out), _stream(stream)))


# ---- adaptive-LayerNorm block (per-image scale / shift / gate) ----------------------------------
MODULATION_NAMES = ("shift1", "scale1", "gate1", "shift2", "scale2", "gate2")


class _BlockModulation(C.Structure):
    _fields_ = [(n, _vp) for n in MODULATION_NAMES]


_lib.nova_pruned_block_forward_adaln.argtypes = [_vp, C.POINTER(_BlockWeights), C.POINTER(_BlockModulation),
                                                 C.POINTER(_BlockShape), _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _i, _vp]
_lib.nova_pruned_block_forward_adaln.restype = _i


def nova_pruned_block_forward_adaln(ctx: Context, w: BlockWeights, modulation: dict, shape: BlockShape, x_in,
                                    keep_idx, cu_keep, k_cache, v_cache, kv_len, append_kv, y_kept,
                                    m_on_device: bool = False, stream=None):
    """nova_pruned_block_forward with per-image modulation: `modulation` maps names from
    MODULATION_NAMES to device bf16 tensors [B, C] (a missing name or None = no such term)."""
    ptrs = []
    for n in MODULATION_NAMES:
        t = modulation.get(n) if modulation else None
        if t is not None:
            assert t.dtype == torch.bfloat16 and t.shape == (shape.B, shape.C)
        ptrs.append(_ptr(t))
    cm = _BlockModulation(*ptrs)
    c = shape._c()
    ctx.check(_lib.nova_pruned_block_forward_adaln(
        ctx.handle, C.byref(w.c), C.byref(cm), C.byref(c), _ptr(x_in), _ptr(keep_idx), _ptr(cu_keep), _ptr(k_cache),
        _ptr(v_cache), _ptr(kv_len), int(bool(append_kv)), _ptr(y_kept), int(bool(m_on_device)), _stream(stream)))


# ---- Eq. 14 + Eq. 15-16 of one layer in one call ---------------------------------------------------
_lib.nova_pruned_layer_forward.argtypes = [_vp, C.POINTER(_BlockWeights), C.POINTER(_BlockModulation),
                                           C.POINTER(_BlockShape), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp,
                                           _i, _i, _i, _i, _vp, _vp, _i, _vp]
_lib.nova_pruned_layer_forward.restype = _i


def nova_pruned_layer_forward(ctx: Context, w: BlockWeights, modulation, shape: BlockShape, x_in, keep_idx, prune_idx,
                              cu_keep, k_cache, v_cache, kv_len, append_kv, cache_prev, h, w_tokens, x_out,
                              cache_out=None, m_on_device: bool = False, stream=None):
    """The block on the kept rows and the restore of the pruned rows in one call: the block's last GEMM
    writes the kept rows of x_out / cache_out directly (no compacted y_kept); results are bit-identical
    to nova_pruned_block_forward[_adaln] followed by nova_restore_from_cache."""
    ptrs = []
    for n in MODULATION_NAMES:
        t = modulation.get(n) if modulation else None
        if t is not None:
            assert t.dtype == torch.bfloat16 and t.shape == (shape.B, shape.C)
        ptrs.append(_ptr(t))
    cm = _BlockModulation(*ptrs)
    c = shape._c()
    assert x_in.shape == (shape.B, shape.N, shape.C) and h * w_tokens == shape.N
    hp, wp = (cache_prev.shape[1], cache_prev.shape[2]) if cache_prev is not None else (0, 0)
    ctx.check(_lib.nova_pruned_layer_forward(
        ctx.handle, C.byref(w.c), C.byref(cm) if modulation else None, C.byref(c), _ptr(x_in), _ptr(keep_idx),
        _ptr(prune_idx), _ptr(cu_keep), _ptr(k_cache), _ptr(v_cache), _ptr(kv_len), int(bool(append_kv)),
        _ptr(cache_prev), hp, wp, h, w_tokens, _ptr(x_out), _ptr(cache_out), int(bool(m_on_device)), _stream(stream)))


# ---- alternative selection scores ------------------------------------------------------------------
_lib.nova_score_mse.argtypes = [_vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp]
_lib.nova_score_mse.restype = _i
_lib.nova_score_attention_mass.argtypes = [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _vp]
_lib.nova_score_attention_mass.restype = _i


def nova_score_mse(ctx: Context, x, ref_prev, h, w, score, stream=None):
    """x [B, h*w, C] bf16, ref_prev [B, hp, wp, C] bf16 -> score [B, h*w] f32: mean squared distance to
    the bilinear resize of the previous scale's map."""
    B, N, Cc = x.shape
    assert N == h * w and ref_prev.shape[0] == B and ref_prev.shape[3] == Cc
    assert x.dtype == torch.bfloat16 and ref_prev.dtype == torch.bfloat16 and score.dtype == torch.float32
    ctx.check(_lib.nova_score_mse(ctx.handle, _ptr(x), _ptr(ref_prev), B, ref_prev.shape[1], ref_prev.shape[2], h, w,
                                  Cc, _ptr(score), _stream(stream)))


def nova_score_attention_mass(ctx: Context, q, k, k_cache, kv_len, n_heads, score, stream=None):
    """q, k [B, N, C] bf16; k_cache [B, Lmax, C] bf16 and kv_len int32 [B] (device) or None, None ->
    score [B, N] f32: share of the scale's attention landing on each token's key."""
    B, N, Cc = q.shape
    assert k.shape == q.shape and q.dtype == torch.bfloat16 and k.dtype == torch.bfloat16
    assert score.dtype == torch.float32 and score.numel() == B * N
    Lmax = k_cache.shape[1] if k_cache is not None else 0
    lse = torch.empty((B, n_heads, N), dtype=torch.float32, device=q.device)
    ctx.check(_lib.nova_score_attention_mass(ctx.handle, _ptr(q), _ptr(k), _ptr(k_cache), _ptr(kv_len), B, N, Cc,
                                             n_heads, Lmax, _ptr(lse), _ptr(score), _stream(stream)))


# ---- block with rotary embedding, QK normalisation, cross-attention ----------------------------------
EXTRA_NAMES = ("rope_cos", "rope_sin", "qk_gain_q", "qk_gain_k", "lnc_g", "lnc_b", "w_q2", "b_q2", "w_o2", "b_o2",
               "cond_k", "cond_v", "cond_len")


class _BlockExtras(C.Structure):
    _fields_ = [("rope_cos", _vp), ("rope_sin", _vp), ("qk_gain_q", _vp), ("qk_gain_k", _vp), ("qk_eps", C.c_float)] + \
               [(n, _vp) for n in ("lnc_g", "lnc_b", "w_q2", "b_q2", "w_o2", "b_o2", "cond_k", "cond_v", "cond_len")] + \
               [("Lc_max", _i)]


_lib.nova_pruned_block_forward_ext.argtypes = [_vp, C.POINTER(_BlockWeights), C.POINTER(_BlockModulation),
                                               C.POINTER(_BlockExtras), C.POINTER(_BlockShape), _vp, _vp, _vp, _vp, _vp,
                                               _vp, _i, _vp, _i, _vp]
_lib.nova_pruned_block_forward_ext.restype = _i


def nova_pruned_block_forward_ext(ctx: Context, w: BlockWeights, modulation, extras: dict, shape: BlockShape, x_in,
                                  keep_idx, cu_keep, k_cache, v_cache, kv_len, append_kv, y_kept,
                                  m_on_device: bool = False, qk_eps: float = 1e-12, stream=None):
    """nova_pruned_block_forward with the optional parts of the text-conditioned backbones. extras maps
    names from EXTRA_NAMES to device tensors (missing or None = absent): rope_cos / rope_sin f32 [N, dh/2];
    qk_gain_q / qk_gain_k bf16 [C]; lnc_g, lnc_b, b_q2, b_o2 bf16 [C], w_q2, w_o2 bf16 [C, C], cond_k / cond_v
    bf16 [B, Lc_max, C], cond_len int32 [B] for the cross-attention."""
    e = {n: (extras.get(n) if extras else None) for n in EXTRA_NAMES}
    dh = shape.C // shape.n_heads
    for n in ("rope_cos", "rope_sin"):
        assert e[n] is None or (e[n].dtype == torch.float32 and e[n].shape == (shape.N, dh // 2))
    Lc = e["cond_k"].shape[1] if e["cond_k"] is not None else 0
    ce = _BlockExtras(_ptr(e["rope_cos"]), _ptr(e["rope_sin"]), _ptr(e["qk_gain_q"]), _ptr(e["qk_gain_k"]), qk_eps,
                      *[_ptr(e[n]) for n in ("lnc_g", "lnc_b", "w_q2", "b_q2", "w_o2", "b_o2", "cond_k", "cond_v", "cond_len")],
                      Lc)
    ptrs = []
    for n in MODULATION_NAMES:
        t = modulation.get(n) if modulation else None
        ptrs.append(_ptr(t))
    cm = _BlockModulation(*ptrs)
    c = shape._c()
    ctx.check(_lib.nova_pruned_block_forward_ext(
        ctx.handle, C.byref(w.c), C.byref(cm) if modulation else None, C.byref(ce), C.byref(c), _ptr(x_in), _ptr(keep_idx),
        _ptr(cu_keep), _ptr(k_cache), _ptr(v_cache), _ptr(kv_len), int(bool(append_kv)), _ptr(y_kept),
        int(bool(m_on_device)), _stream(stream)))

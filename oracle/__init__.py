"""CPU oracle of the NOVA pruned-scale step (test infrastructure, not product).

This package wraps ``nova_oracle.cpp`` (plain C++, double accumulators, written
from the paper's equations) for the tests, the smoke check and the benchmark's
CPU-baseline leg. Nothing in the CUDA library or its Python binding may import
it, and it imports nothing from them.

All arrays are numpy; floating tensors are float32 (bf16 inputs must be widened
by the caller), index tensors int32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nova_oracle.cpp")
_LIB = os.path.join(_HERE, "libnova_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, OpenMP over rows). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["g++", "-O2", "-fopenmp", "-std=c++17", "-shared", "-fPIC", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _SchedParams(ctypes.Structure):
    _fields_ = [
        ("t_est", ctypes.c_int),
        ("alpha", ctypes.c_double),
        ("tau", ctypes.c_double),
        ("lam", ctypes.c_double),
        ("k_min", ctypes.c_int),
        ("ratio_max", ctypes.c_double),
        ("force_act_scale", ctypes.c_int),
        ("force_keep_ratio", ctypes.c_double),
    ]


class _BlockWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in (
        "ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
        "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")] + [("eps", ctypes.c_float)]


MODULATION_NAMES = ("shift1", "scale1", "gate1", "shift2", "scale2", "gate2")


class _BlockModulation(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in MODULATION_NAMES]


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def scale_entropy(logits: np.ndarray):
    """Eq. 4 and Eq. 7. logits [S, N, V] -> (ent [S, N] f32, mean [S] f32)."""
    z = _f32(logits)
    S, N, V = z.shape
    ent = np.empty((S, N), np.float32)
    mean = np.empty((S,), np.float32)
    _load().oracle_scale_entropy(_p(z), S, N, V, _p(ent), _p(mean))
    return ent, mean


def head_entropy(x: np.ndarray, w: np.ndarray, b=None):
    """Eq. 4 / Eq. 7 on the codebook head's output: logits = x @ w.T + b, never rounded.
    x [S, N, C], w [V, C], b [V] or None -> (ent [S, N] f32, mean [S] f32)."""
    x = _f32(x)
    w = _f32(w)
    S, N, C = x.shape
    V = w.shape[0]
    assert w.shape == (V, C)
    bb = _f32(b) if b is not None else None
    ent = np.empty((S, N), np.float32)
    mean = np.empty((S,), np.float32)
    _load().oracle_head_entropy(_p(x), _p(w), _p(bb) if bb is not None else None, S, N, C, V, _p(ent), _p(mean))
    return ent, mean


@dataclass
class SchedParams:
    """Hyper-parameters of Eq. 9-11 (paper defaults) plus this build's clamps and overrides."""
    t_est: int = 5
    alpha: float = 0.5
    tau: float = 0.8
    lam: float = 0.1
    k_min: int = 1
    ratio_max: float = 1.0
    force_act_scale: int = 0
    force_keep_ratio: float = -1.0


def keep_ratios(p: SchedParams, t: int, j: int, N_t: int, hbar_scale, hbar_layer=None):
    """Eq. 8-13 and the keep count.

    hbar_scale [B, t] (scales 1..t), hbar_layer [B, j] (layers 1..j of scale t) or None
    when j == 1. Returns dict(t_star, act_scale, ratio_scale, ratio_layer, keep).
    """
    hs = _f32(hbar_scale)
    B = hs.shape[0]
    assert hs.shape == (B, t)
    hl = _f32(hbar_layer) if hbar_layer is not None else np.zeros((B, max(j, 1)), np.float32)
    assert hl.shape == (B, max(j, 1))
    cp = _SchedParams(p.t_est, p.alpha, p.tau, p.lam, p.k_min, p.ratio_max,
                      p.force_act_scale, p.force_keep_ratio)
    t_star = np.zeros(B, np.int32)
    act = np.zeros(B, np.int32)
    rs = np.zeros(B, np.float64)
    rl = np.zeros(B, np.float64)
    keep = np.zeros(B, np.int32)
    _load().oracle_keep_ratios(ctypes.byref(cp), B, t, j, N_t, _p(hs), _p(hl),
                               _p(t_star), _p(act), _p(rs), _p(rl), _p(keep))
    return dict(t_star=t_star, act_scale=act, ratio_scale=rs, ratio_layer=rl, keep=keep)


def select_topk(ent: np.ndarray, k):
    """Keep the k[s] highest entropies of each segment, ties to the lower index.

    ent [S, N] -> (keep_idx [sum k], prune_idx [S*N - sum k], cu_keep [S+1], pos [S, N]).
    """
    e = _f32(ent)
    S, N = e.shape
    kk = _i32(k)
    assert kk.shape == (S,) and (kk >= 0).all() and (kk <= N).all()
    M = int(kk.sum())
    keep_idx = np.empty(M, np.int32)
    prune_idx = np.empty(S * N - M, np.int32)
    cu = np.empty(S + 1, np.int32)
    pos = np.empty((S, N), np.int32)
    _load().oracle_select_topk(_p(e), S, N, _p(kk), _p(keep_idx), _p(prune_idx), _p(cu), _p(pos))
    return keep_idx, prune_idx, cu, pos


WEIGHT_NAMES = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
                "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")


def pruned_block_forward(weights: dict, eps: float, n_heads: int, x_in, keep_idx, cu_keep,
                         k_cache, v_cache, kv_len, rows=None, modulation=None):
    """Eq. 14 on the kept tokens (pre-LN block; keys = cache ++ kept tokens' own k/v).

    x_in [B, N, C]; k_cache/v_cache [B, Lmax, C]; kv_len [B]; rows: optional compacted
    row numbers to evaluate. modulation: optional dict of per-image [B, C] arrays named in
    MODULATION_NAMES (adaptive LayerNorm: LN output * (1 + scale) + shift, branch * gate); a
    missing name means no such term. Returns (y [R, C], k_new [M, C], v_new [M, C]).
    """
    x = _f32(x_in)
    B, N, C = x.shape
    w = {n: _f32(weights[n]) for n in WEIGHT_NAMES}
    F = w["w_fc1"].shape[0]
    assert w["w_qkv"].shape == (3 * C, C) and w["w_fc2"].shape == (C, F)
    ki, cu = _i32(keep_idx), _i32(cu_keep)
    M = int(cu[B])
    kc, vc = _f32(k_cache), _f32(v_cache)
    Lmax = kc.shape[1]
    assert kc.shape == (B, Lmax, C) and vc.shape == kc.shape
    kl = _i32(kv_len)
    rr = _i32(rows) if rows is not None else None
    R = len(rr) if rr is not None else M
    y = np.empty((R, C), np.float32)
    k_new = np.empty((M, C), np.float32)
    v_new = np.empty((M, C), np.float32)
    cw = _BlockWeights(*[_p(w[n]) for n in WEIGHT_NAMES], eps)
    if modulation is None:
        _load().oracle_pruned_block_forward(
            ctypes.byref(cw), B, N, C, n_heads, F, Lmax, _p(x), _p(ki), _p(cu),
            _p(kc), _p(vc), _p(kl), _p(rr), R, _p(y), _p(k_new), _p(v_new))
        return y, k_new, v_new
    md = {n: _f32(modulation[n]) for n in MODULATION_NAMES if modulation.get(n) is not None}
    for a in md.values():
        assert a.shape == (B, C)
    cm = _BlockModulation(*[_p(md[n]) if n in md else None for n in MODULATION_NAMES])
    _load().oracle_pruned_block_forward_mod(
        ctypes.byref(cw), ctypes.byref(cm), B, N, C, n_heads, F, Lmax, _p(x), _p(ki), _p(cu),
        _p(kc), _p(vc), _p(kl), _p(rr), R, _p(y), _p(k_new), _p(v_new))
    return y, k_new, v_new


EXT_NAMES = ("rope_cos", "rope_sin", "qk_gain_q", "qk_gain_k", "lnc_g", "lnc_b", "w_q2", "b_q2", "w_o2", "b_o2", "ck", "cv")


class _BlockExt(ctypes.Structure):
    _fields_ = [("rope_cos", ctypes.c_void_p), ("rope_sin", ctypes.c_void_p), ("qk_gain_q", ctypes.c_void_p),
                ("qk_gain_k", ctypes.c_void_p), ("qk_eps", ctypes.c_float)] + \
               [(n, ctypes.c_void_p) for n in ("lnc_g", "lnc_b", "w_q2", "b_q2", "w_o2", "b_o2", "ck", "cv", "cond_len")] + \
               [("Lc_max", ctypes.c_int)]


def pruned_block_forward_ext(weights: dict, eps: float, n_heads: int, x_in, keep_idx, cu_keep, k_cache, v_cache, kv_len,
                             ext: dict, rows=None, modulation=None, qk_eps: float = 1e-12):
    """pruned_block_forward with the optional parts of the text-conditioned backbones. ext maps names
    from EXT_NAMES to arrays (missing = absent): rope_cos / rope_sin [N, dh/2]; qk_gain_q / qk_gain_k [C];
    lnc_g, lnc_b [C], w_q2, w_o2 [C, C], b_q2, b_o2 [C], ck, cv [B, Lc_max, C] together with
    ext["cond_len"] int32 [B] for the cross-attention. Returns (y, k_new, v_new); k_new holds the
    transformed keys."""
    x = _f32(x_in)
    B, N, C = x.shape
    w = {n: _f32(weights[n]) for n in WEIGHT_NAMES}
    F = w["w_fc1"].shape[0]
    ki, cu = _i32(keep_idx), _i32(cu_keep)
    M = int(cu[B])
    kc, vc = _f32(k_cache), _f32(v_cache)
    Lmax = kc.shape[1]
    kl = _i32(kv_len)
    rr = _i32(rows) if rows is not None else None
    R = len(rr) if rr is not None else M
    y = np.empty((R, C), np.float32)
    k_new = np.empty((M, C), np.float32)
    v_new = np.empty((M, C), np.float32)
    cw = _BlockWeights(*[_p(w[n]) for n in WEIGHT_NAMES], eps)
    e = {n: _f32(ext[n]) for n in EXT_NAMES if ext.get(n) is not None}
    dh = C // n_heads
    if "rope_cos" in e:
        assert e["rope_cos"].shape == (N, dh // 2) and e["rope_sin"].shape == (N, dh // 2)
    cl = _i32(ext["cond_len"]) if ext.get("cond_len") is not None else None
    Lc = e["ck"].shape[1] if "ck" in e else 0
    if "w_q2" in e:
        assert cl is not None and e["ck"].shape == (B, Lc, C) and e["cv"].shape == (B, Lc, C)
    g = lambda n: _p(e[n]) if n in e else None
    ce = _BlockExt(g("rope_cos"), g("rope_sin"), g("qk_gain_q"), g("qk_gain_k"), qk_eps, g("lnc_g"), g("lnc_b"),
                   g("w_q2"), g("b_q2"), g("w_o2"), g("b_o2"), g("ck"), g("cv"), _p(cl) if cl is not None else None, Lc)
    cm = None
    md = {}
    if modulation is not None:
        md = {n: _f32(modulation[n]) for n in MODULATION_NAMES if modulation.get(n) is not None}
        cm = _BlockModulation(*[_p(md[n]) if n in md else None for n in MODULATION_NAMES])
    _load().oracle_pruned_block_forward_ext(
        ctypes.byref(cw), ctypes.byref(cm) if cm is not None else None, ctypes.byref(ce), B, N, C, n_heads, F, Lmax,
        _p(x), _p(ki), _p(cu), _p(kc), _p(vc), _p(kl), _p(rr), R, _p(y), _p(k_new), _p(v_new))
    return y, k_new, v_new


def restore_from_cache(x_in, y_kept, keep_idx, prune_idx, cu_keep, cache_prev, h, w,
                       want_cache=True):
    """Eq. 15-16. x_in [B, h*w, C]; y_kept [M, C]; cache_prev [B, hp, wp, C].

    Returns (x_out [B, h*w, C], cache_out [B, h*w, C] or None).
    """
    x = _f32(x_in)
    B, N, C = x.shape
    assert N == h * w
    cp = _f32(cache_prev)
    _, hp, wp, _ = cp.shape
    y = _f32(y_kept)
    ki, pi, cu = _i32(keep_idx), _i32(prune_idx), _i32(cu_keep)
    x_out = np.empty_like(x)
    cache_out = np.empty_like(x) if want_cache else None
    _load().oracle_restore_from_cache(_p(x), _p(y), _p(ki), _p(pi), _p(cu), _p(cp),
                                      hp, wp, h, w, C, B, _p(x_out), _p(cache_out))
    return x_out, cache_out


def score_mse(x, ref_prev, h: int, w: int):
    """MSE selection score (reading of the paper's selection-metric ablation): mean squared distance
    between a token and the bilinear resize of the previous scale's map to its position.
    x [B, h*w, C], ref_prev [B, hp, wp, C] -> score [B, h*w] f32."""
    xx, rr = _f32(x), _f32(ref_prev)
    B, N, C = xx.shape
    assert N == h * w and rr.shape[0] == B and rr.shape[3] == C
    score = np.empty((B, N), np.float32)
    _load().oracle_score_mse(_p(xx), _p(rr), B, rr.shape[1], rr.shape[2], h, w, C, _p(score))
    return score


def score_attention_mass(q, k, k_cache, kv_len, n_heads: int):
    """Attention-mass selection score: the share of the scale's attention (all N tokens as queries,
    keys = prior cache rows followed by the N tokens' own keys) that lands on each token's key,
    averaged over heads and queries. q, k [B, N, C]; k_cache [B, Lmax, C] or None; kv_len [B] or None
    -> score [B, N] f32."""
    qq, kk = _f32(q), _f32(k)
    B, N, C = qq.shape
    kc = _f32(k_cache) if k_cache is not None else None
    kl = _i32(kv_len) if kv_len is not None else np.zeros(B, np.int32)
    Lmax = kc.shape[1] if kc is not None else 0
    assert kc is not None or (kl == 0).all()
    score = np.empty((B, N), np.float32)
    _load().oracle_score_attention_mass(_p(qq), _p(kk), _p(kc) if kc is not None else None, _p(kl), B, N, C, n_heads,
                                        Lmax, _p(score))
    return score

"""Seeded synthetic inputs with the shapes and statistics of VAR-style workloads.

This module only draws random tensors and lays out shapes. It contains none of the
method's arithmetic (no entropy, ratio, selection, block or restore computation) and
is the one piece shared by the CUDA-path tests, the CPU oracle tests and the bench:
both sides receive the same bytes.

All floating tensors are returned as torch tensors (bf16 unless stated) on the
requested device; a given (seed, device type) pair always yields the same values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

V_CODEBOOK = 4096


@dataclass(frozen=True)
class ModelShape:
    name: str
    L: int            # transformer layers
    C: int            # width
    heads: int
    F: int            # MLP hidden width
    scales: tuple     # side length of every scale
    B: int            # batch (images)

    @property
    def dh(self) -> int:
        return self.C // self.heads

    def tokens(self, t: int) -> int:
        """Tokens of scale t (1-based)."""
        return self.scales[t - 1] ** 2

    def prior_tokens(self, t: int) -> int:
        return sum(s * s for s in self.scales[: t - 1])

    @property
    def total_tokens(self) -> int:
        return sum(s * s for s in self.scales)


# The five workload shapes (batch and scale schedules as in the benchmark configs).
CONFIGS = {
    "c1_single_step": ModelShape("c1_single_step", 1, 1024, 16, 4096,
                                 (1, 2, 3, 4, 5, 6, 8, 10, 13, 16), 2),
    "c2_var_d16_256": ModelShape("c2_var_d16_256", 16, 1024, 16, 4096,
                                 (1, 2, 3, 4, 5, 6, 8, 10, 13, 16), 8),
    "c3_var_d30_512": ModelShape("c3_var_d30_512", 30, 1920, 30, 7680,
                                 (1, 2, 3, 4, 6, 9, 13, 18, 24, 32), 4),
    "c4_1024": ModelShape("c4_1024", 32, 2048, 16, 8192,
                          (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64), 4),
    "c5_2048": ModelShape("c5_2048", 32, 2048, 16, 8192,
                          (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64, 80, 96, 128), 1),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def randn_bf16(shape, seed: int, device="cpu", std: float = 1.0, mean: float = 0.0) -> torch.Tensor:
    """N(mean, std^2) drawn in fp32 then rounded to bf16."""
    x = torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return (x * std + mean).to(torch.bfloat16)


def block_weights(C: int, F: int, seed: int, device="cpu") -> dict:
    """Random-init weights of one pre-LN block: N(0, 0.02^2), LN gain 1 + N(0, 0.02^2).

    Matrices are [out, in] row-major.
    """
    s = 0.02
    shapes = {
        "ln1_g": (C,), "ln1_b": (C,), "w_qkv": (3 * C, C), "b_qkv": (3 * C,),
        "w_o": (C, C), "b_o": (C,), "ln2_g": (C,), "ln2_b": (C,),
        "w_fc1": (F, C), "b_fc1": (F,), "w_fc2": (C, F), "b_fc2": (C,),
    }
    out = {}
    for i, (name, shp) in enumerate(shapes.items()):
        mean = 1.0 if name in ("ln1_g", "ln2_g") else 0.0
        out[name] = randn_bf16(shp, seed * 1000 + i, device, std=s, mean=mean)
    return out


def activations(B: int, N: int, C: int, seed: int, device="cpu") -> torch.Tensor:
    """Layer input x_in [B, N, C], N(0, 1)."""
    return randn_bf16((B, N, C), seed, device)


def kv_cache(B: int, Lmax: int, n_valid: int, C: int, seed: int, device="cpu"):
    """Prior-scale K and V caches [B, Lmax, C]; rows >= n_valid are zero."""
    k = torch.zeros((B, Lmax, C), dtype=torch.bfloat16, device=device)
    v = torch.zeros((B, Lmax, C), dtype=torch.bfloat16, device=device)
    if n_valid > 0:
        k[:, :n_valid] = randn_bf16((B, n_valid, C), seed, device)
        v[:, :n_valid] = randn_bf16((B, n_valid, C), seed + 1, device)
    kv_len = torch.full((B,), n_valid, dtype=torch.int32, device=device)
    return k, v, kv_len


def residual_cache(B: int, hp: int, wp: int, C: int, seed: int, device="cpu") -> torch.Tensor:
    """Previous scale's residual cache [B, hp, wp, C], N(0, 1)."""
    return randn_bf16((B, hp, wp, C), seed, device)


# ----------------------------------------------------------------------------------
# Logits: z[b, i, v] = a[b, i] * n[b, i, v], n ~ N(0, 1). The per-token inverse
# temperature a sets how peaked the row is: small a -> near-uniform row, a beyond
# about sqrt(2 ln V) ~ 4.1 -> a row dominated by a few codes.
# ----------------------------------------------------------------------------------
def logits_from_temperature(a: torch.Tensor, V: int, seed: int, dtype=torch.bfloat16) -> torch.Tensor:
    """a [B, N] (fp32, any device) -> logits [B, N, V] on a's device."""
    B, N = a.shape
    n = torch.randn((B, N, V), generator=_gen(seed, a.device), device=a.device, dtype=torch.float32)
    n.mul_(a.to(torch.float32).unsqueeze(-1))
    return n.to(dtype)


def smooth_temperature_field(B: int, h: int, w: int, seed: int, a_lo: float = 0.5,
                             a_hi: float = 6.0, device="cpu") -> torch.Tensor:
    """Smooth spatial field: a few seeded low-frequency cosines, pushed through a steep
    sigmoid around the median so half of the map is near a_lo and half near a_hi.
    Returns a [B, h*w] fp32.
    """
    g = _gen(seed, "cpu")
    ys = (torch.arange(h, dtype=torch.float64) + 0.5) / h
    xs = (torch.arange(w, dtype=torch.float64) + 0.5) / w
    out = []
    for _ in range(B):
        f = torch.zeros((h, w), dtype=torch.float64)
        for _m in range(4):
            c = torch.rand((), generator=g, dtype=torch.float64) + 0.5
            p = torch.randint(0, 3, (), generator=g).item()
            q = torch.randint(0, 3, (), generator=g).item()
            if p == 0 and q == 0:
                p = 1
            phi = torch.rand((), generator=g, dtype=torch.float64) * 2 * math.pi
            f += c * torch.cos(2 * math.pi * (p * xs[None, :] + q * ys[:, None]) + phi)
        f = f.flatten()
        sd = f.std().clamp_min(1e-9)
        u = torch.sigmoid((f - f.median()) / (0.1 * sd))
        out.append(a_lo + (a_hi - a_lo) * u)
    return torch.stack(out).to(torch.float32).to(device)


def blob_temperature_field(B: int, h: int, w: int, seed: int, cover: float = 0.2,
                           a_in: float = 0.7, a_out: float = 6.0, n_blobs: int = 12,
                           device="cpu") -> torch.Tensor:
    """High-entropy tokens (small a) inside seeded random discs whose union covers
    about `cover` of the map, low entropy elsewhere. Returns a [B, h*w] fp32.
    """
    g = _gen(seed, "cpu")
    ys = ((torch.arange(h, dtype=torch.float64) + 0.5) / h)[:, None]
    xs = ((torch.arange(w, dtype=torch.float64) + 0.5) / w)[None, :]
    out = []
    for _ in range(B):
        cx = torch.rand(n_blobs, generator=g, dtype=torch.float64)
        cy = torch.rand(n_blobs, generator=g, dtype=torch.float64)
        rel = torch.rand(n_blobs, generator=g, dtype=torch.float64) * 0.5 + 0.75
        # grow a common radius factor until the union reaches the requested cover
        lo, hi = 0.0, 1.0
        for _it in range(40):
            mid = 0.5 * (lo + hi)
            inside = torch.zeros((h, w), dtype=torch.bool)
            for i in range(n_blobs):
                inside |= ((xs - cx[i]) ** 2 + (ys - cy[i]) ** 2) <= (mid * rel[i]) ** 2
            if inside.double().mean().item() < cover:
                lo = mid
            else:
                hi = mid
        inside = torch.zeros((h, w), dtype=torch.bool)
        for i in range(n_blobs):
            inside |= ((xs - cx[i]) ** 2 + (ys - cy[i]) ** 2) <= (hi * rel[i]) ** 2
        a = torch.where(inside, torch.tensor(a_in, dtype=torch.float64),
                        torch.tensor(a_out, dtype=torch.float64))
        out.append(a.flatten())
    return torch.stack(out).to(torch.float32).to(device)


def scale_envelope_temperatures(B: int, T: int, seed: int, V: int = V_CODEBOOK,
                                H_lo: float = 4.5, H_hi: float = 8.0):
    """Per-image, per-scale global inverse temperatures a[b, t-1] chosen so that the mean
    row entropy rises with the scale index roughly as a seeded sigmoid
    H_lo + (H_hi - H_lo) * sigmoid((t - t0) / w): for Gaussian logits of standard
    deviation a below the concentration threshold the row entropy is close to
    ln V - a^2 / 2, which is inverted here. t0 in [2.5, 5.5], w in [0.6, 1.5].
    Returns (a [B, T] fp32, target_H [B, T] fp32).
    """
    g = _gen(seed, "cpu")
    t0 = 2.5 + 3.0 * torch.rand(B, generator=g, dtype=torch.float64)
    wd = 0.6 + 0.9 * torch.rand(B, generator=g, dtype=torch.float64)
    t = torch.arange(1, T + 1, dtype=torch.float64)[None, :]
    target = H_lo + (H_hi - H_lo) * torch.sigmoid((t - t0[:, None]) / wd[:, None])
    a = torch.sqrt(torch.clamp(2.0 * (math.log(V) - target), min=0.0))
    return a.to(torch.float32), target.to(torch.float32)


def layer_inverse_temperatures(L: int, seed: int) -> torch.Tensor:
    """Per-layer multipliers beta_j in [0.8, 1.25] applied to a scale's logits so that the
    layer mean entropies differ across the L layers. Returns [L] fp32.
    """
    g = _gen(seed, "cpu")
    return (0.8 + 0.45 * torch.rand(L, generator=g, dtype=torch.float64)).to(torch.float32)


def to_f32_numpy(t: torch.Tensor):
    """Exact widening of a (bf16/fp32) tensor to a float32 numpy array on the host."""
    return t.detach().to("cpu", torch.float32).contiguous().numpy()

"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every symbol the
header declares, and its host-side schedule arithmetic (Eq. 8-13) is bit-identical to the
oracle's on random histories."""
import ctypes
import os
import re

import numpy as np
import torch

import oracle
import paper_2602_01345_b200 as nova

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "nova.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nova_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert {"nova_scale_entropy", "nova_keep_ratios", "nova_select_topk",
            "nova_pruned_block_forward", "nova_restore_from_cache"} <= set(names)
    lib = ctypes.CDLL(nova.lib_path())
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/nova.h but not exported"


def test_status_strings_and_default_params():
    lib = ctypes.CDLL(nova.lib_path())
    lib.nova_status_string.restype = ctypes.c_char_p
    assert lib.nova_status_string(0) == b"ok"
    assert lib.nova_status_string(6) == b"device-side wait expired"
    from paper_2602_01345_b200.binding import _SchedParams
    p = _SchedParams()
    lib.nova_sched_params_default(ctypes.byref(p))
    assert (p.t_est, p.alpha, p.tau, p.lam, p.k_min, p.ratio_max, p.force_act_scale) == (5, 0.5, 0.8, 0.1, 1, 1.0, 0)
    assert p.force_keep_ratio < 0


def test_workspace_bytes_host_side():
    ok = nova.BlockShape(B=2, N=256, C=1024, n_heads=16, F=4096, Lmax=680, M=256)
    need = nova.nova_block_workspace_bytes(ok)
    assert need >= 256 * (4 * 1024 + 4096) * 2
    bad = nova.BlockShape(B=2, N=256, C=1000, n_heads=16, F=4096, Lmax=680, M=256)
    assert nova.nova_block_workspace_bytes(bad) == 0
    bad_dh = nova.BlockShape(B=2, N=256, C=1024, n_heads=32, F=4096, Lmax=680, M=256)   # dh = 32
    assert nova.nova_block_workspace_bytes(bad_dh) == 0


def _compare(p_or, p_lib, t, j, N, hs, hl):
    want = oracle.keep_ratios(p_or, t, j, N, hs, hl)
    got = nova.nova_keep_ratios(p_lib, t, j, N, torch.from_numpy(hs), torch.from_numpy(hl) if hl is not None else None)
    for key in ("t_star", "act_scale", "keep"):
        assert np.array_equal(got[key].numpy(), want[key]), key
    for key in ("ratio_scale", "ratio_layer"):
        assert np.array_equal(got[key].numpy(), want[key]), key     # bit-identical doubles


def test_keep_ratios_bit_exact_against_oracle_random_histories():
    rng = np.random.default_rng(0)
    for trial in range(300):
        B = int(rng.integers(1, 9))
        T = int(rng.integers(1, 17))
        L = int(rng.integers(1, 33))
        N = int(rng.choice([1, 7, 256, 1024, 4096, 16384]))
        # rising-then-flattening curves with noise so every branch of the trigger is visited
        t_axis = np.arange(1, T + 1)
        t0 = rng.uniform(1, 8, (B, 1))
        hs = (2 + 6 / (1 + np.exp(-(t_axis[None] - t0) / rng.uniform(0.4, 2, (B, 1)))) +
              0.05 * rng.standard_normal((B, T))).astype(np.float32)
        j = int(rng.integers(1, L + 1))
        hl = (hs[:, -1:] * rng.uniform(0.7, 1.3, (B, j))).astype(np.float32)
        kw = dict(t_est=int(rng.integers(2, 7)), alpha=float(rng.uniform(0.1, 0.9)),
                  tau=float(rng.uniform(0.3, 2.0)), lam=float(rng.uniform(0, 0.3)),
                  k_min=int(rng.integers(0, 4)), ratio_max=float(rng.uniform(0.5, 1.0)))
        if trial % 5 == 0:
            kw["force_act_scale"] = int(rng.integers(1, T + 2))
        if trial % 7 == 0:
            kw["force_keep_ratio"] = float(rng.choice([0.2, 0.25, 0.5, 0.75, 1.0]))
        _compare(oracle.SchedParams(**kw), nova.SchedParams(**kw), T, j, N, hs, hl)


def test_keep_ratios_all_layers_equals_layer_by_layer_and_oracle():
    """The all-layers call gives, for every layer j, what the per-layer call and the oracle give on
    the means of layers 1..j (Eq. 12-13), bit for bit."""
    rng = np.random.default_rng(3)
    for trial in range(40):
        B, T, L = int(rng.integers(1, 9)), int(rng.integers(6, 14)), int(rng.integers(1, 33))
        N = int(rng.choice([256, 1024, 4096]))
        t_axis = np.arange(1, T + 1)
        hs = (2 + 6 / (1 + np.exp(-(t_axis[None] - rng.uniform(1, 6, (B, 1))) / rng.uniform(0.4, 2, (B, 1)))) +
              0.05 * rng.standard_normal((B, T))).astype(np.float32)
        hl = (hs[:, -1:] * rng.uniform(0.7, 1.3, (B, L))).astype(np.float32)
        kw = dict(lam=float(rng.uniform(0, 0.3)), tau=float(rng.uniform(0.3, 2.0)))
        if trial % 4 == 0:
            kw["force_act_scale"] = T - 1
        got = nova.nova_keep_ratios_layers(nova.SchedParams(**kw), T, N, torch.from_numpy(hs), torch.from_numpy(hl))
        pruned = 0
        for j in range(1, L + 1):
            want = oracle.keep_ratios(oracle.SchedParams(**kw), T, j, N, hs, hl[:, :j].copy())
            assert np.array_equal(got["keep"][j - 1].numpy(), want["keep"]), (trial, j)
            assert np.array_equal(got["ratio_layer"][j - 1].numpy(), want["ratio_layer"]), (trial, j)
            pruned += int((want["keep"] < N).sum())
        assert np.array_equal(got["t_star"].numpy(), want["t_star"])
        assert np.array_equal(got["act_scale"].numpy(), want["act_scale"])
        assert np.array_equal(got["ratio_scale"].numpy(), want["ratio_scale"])
        if trial % 4 == 0:
            assert pruned > 0


def test_keep_ratios_worked_example_and_errors():
    hs = np.array([[1, 2, 3, 4, 5, 6, 6, 6, 6, 6]], np.float32)
    got = nova.nova_keep_ratios(nova.SchedParams(), 8, 1, 256, torch.from_numpy(hs[:, :8]))
    assert got["t_star"].item() == 7 and got["act_scale"].item() == 8 and got["keep"].item() == 128
    import pytest
    with pytest.raises(nova.NovaError):
        nova.nova_keep_ratios(nova.SchedParams(tau=0.0), 8, 1, 256, torch.from_numpy(hs[:, :8]))
    with pytest.raises(nova.NovaError):
        nova.nova_keep_ratios(nova.SchedParams(t_est=1), 8, 1, 256, torch.from_numpy(hs[:, :8]))

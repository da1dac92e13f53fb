"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here touches the CUDA path. Each test checks the oracle against a closed form,
an invariant, a library routine it does not itself call (numpy/scipy/torch fp64), or
brute force on tiny inputs, chosen so that a plausible slip in the oracle (dropped term,
wrong sign or index, transposed operand) fails at least one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as TF

import oracle

V = 4096
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ entropy (Eq. 4, 7)
def test_entropy_uniform_is_ln_v():
    z = np.full((1, 3, V), 0.37, np.float32)
    ent, mean = oracle.scale_entropy(z)
    assert np.allclose(ent, math.log(V), atol=1e-6)
    assert abs(mean[0] - math.log(V)) < 1e-6
    assert abs(math.log(V) - 8.317766) < 1e-6


def test_entropy_one_hot_is_zero():
    z = np.zeros((1, 2, V), np.float32)
    z[0, 0, 17] = 1000.0          # exp(-1000) underflows to 0 in double: exactly 0
    z[0, 1, 4095] = 100.0         # 4095 * e^-100 * ~100: far below fp32 resolution of 1
    ent, _ = oracle.scale_entropy(z)
    assert ent[0, 0] == 0.0
    assert 0.0 <= ent[0, 1] < 1e-30


def test_entropy_two_level_closed_form():
    # m logits at value a, V-m at value b
    for m, a, b in [(1, 3.0, 0.0), (100, 2.0, -1.0), (4000, -0.5, 0.25), (7, 9.0, 1.0)]:
        z = np.full((1, 1, V), b, np.float32)
        z[0, 0, :m] = a
        Z = m * math.exp(a) + (V - m) * math.exp(b)
        want = math.log(Z) - (m * a * math.exp(a) + (V - m) * b * math.exp(b)) / Z
        ent, _ = oracle.scale_entropy(z)
        assert abs(ent[0, 0] - want) < 1e-6 * max(1.0, want)


def test_entropy_binary_matches_sigmoid_entropy():
    z = np.array([[[0.3, -1.2]], [[5.0, 5.0]], [[-2.0, 4.0]]], np.float32)  # V = 2
    ent, _ = oracle.scale_entropy(z)
    for r in range(3):
        p = 1.0 / (1.0 + math.exp(-(float(z[r, 0, 1]) - float(z[r, 0, 0]))))
        want = -(p * math.log(p) + (1 - p) * math.log(1 - p))
        assert abs(ent[r, 0] - want) < 1e-6


def test_entropy_shift_invariance_bounds_and_library():
    from scipy.special import softmax
    from scipy.stats import entropy as sp_entropy
    rng = np.random.default_rng(0)
    z = (rng.standard_normal((2, 5, 512)) * rng.uniform(0.2, 6.0, (2, 5, 1))).astype(np.float32)
    ent, mean = oracle.scale_entropy(z)
    ent_shift, _ = oracle.scale_entropy(z + np.float32(8.0))   # exact shift in fp32 for these magnitudes? use tolerance
    assert np.allclose(ent, ent_shift, atol=2e-5)
    assert (ent >= 0).all() and (ent <= math.log(512) + 1e-6).all()
    lib = sp_entropy(softmax(z.astype(np.float64), axis=-1), axis=-1)
    assert np.allclose(ent, lib, atol=1e-6)
    assert np.allclose(mean, lib.mean(axis=1), atol=1e-6)


def test_entropy_neg_inf_logit_contributes_nothing():
    z = np.zeros((1, 1, 8), np.float32)
    z[0, 0, 4:] = -np.inf
    ent, _ = oracle.scale_entropy(z)
    assert abs(ent[0, 0] - math.log(4)) < 1e-7


# ----------------------------------------------------------- entropy of the codebook head
def test_head_entropy_closed_forms():
    """Zero head -> uniform -> ln V; bias only -> entropy of softmax(b) (two-level closed form);
    a head whose rows are +-a along one hidden unit -> two-level distribution set by x."""
    S, N, C, V = 1, 3, 8, 64
    x = np.random.default_rng(0).standard_normal((S, N, C)).astype(np.float32)
    ent, mean = oracle.head_entropy(x, np.zeros((V, C), np.float32))
    assert np.allclose(ent, math.log(V), atol=1e-6) and np.allclose(mean, math.log(V), atol=1e-6)
    b = np.zeros(V, np.float32)
    b[:5] = 2.0
    ent, _ = oracle.head_entropy(x, np.zeros((V, C), np.float32), b)
    Z = 5 * math.exp(2.0) + (V - 5)
    assert np.allclose(ent, math.log(Z) - 5 * 2.0 * math.exp(2.0) / Z, atol=1e-6)
    w = np.zeros((V, C), np.float32)
    w[: V // 2, 3] = 1.0                    # half of the codes see +x_3, the other half 0
    ent, _ = oracle.head_entropy(x, w)
    for i in range(N):
        a = float(x[0, i, 3])
        Z = (V // 2) * math.exp(a) + V // 2
        want = math.log(Z) - (V // 2) * a * math.exp(a) / Z
        assert abs(ent[0, i] - want) < 1e-6


def test_head_entropy_equals_entropy_of_library_matmul_and_operand_order():
    """Against numpy's float64 matmul followed by scipy's softmax entropy; a transposed or
    mis-strided weight would fail (V != C, random values), so would a dropped bias."""
    rng = np.random.default_rng(3)
    S, N, C, V = 2, 5, 24, 40
    x = rng.standard_normal((S, N, C)).astype(np.float32)
    w = (0.3 * rng.standard_normal((V, C))).astype(np.float32)
    b = rng.standard_normal(V).astype(np.float32)
    ent, mean = oracle.head_entropy(x, w, b)
    from scipy.special import softmax
    from scipy.stats import entropy as sp_entropy
    z = x.astype(np.float64) @ w.astype(np.float64).T + b.astype(np.float64)
    want = sp_entropy(softmax(z, axis=-1), axis=-1)
    assert np.abs(ent - want).max() < 1e-6
    assert np.abs(mean - want.mean(axis=1)).max() < 1e-6
    ent_nb, _ = oracle.head_entropy(x, w)
    assert np.abs(ent_nb - want).max() > 1e-3          # the bias matters in this example
    # and it is the same function as scale_entropy on the unrounded logits
    ent2, _ = oracle.scale_entropy(z.astype(np.float32))
    assert np.abs(ent - ent2).max() < 1e-5


def test_mean_is_per_segment_and_permutation_invariant():
    rng = np.random.default_rng(1)
    z = rng.standard_normal((3, 16, 64)).astype(np.float32) * 3
    ent, mean = oracle.scale_entropy(z)
    perm = rng.permutation(16)
    ent_p, mean_p = oracle.scale_entropy(z[:, perm])
    assert np.array_equal(ent[:, perm], ent_p)
    assert np.allclose(mean, mean_p, atol=1e-6)
    assert np.allclose(mean, ent.astype(np.float64).mean(axis=1), atol=1e-6)


# ------------------------------------------------------- trigger and ratios (Eq. 8-13)
def _read_golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=")
                vals[k.strip()] = v.strip()
    return vals


def test_schedule_worked_example_golden():
    gold = _read_golden("schedule_worked_example.txt")
    hbar = np.array([[float(x) for x in gold["hbar"].split()]], np.float32)
    p = oracle.SchedParams()
    assert (p.t_est, p.alpha, p.tau, p.lam) == (5, 0.5, 0.8, 0.1)   # paper's hyper-parameters
    for t in range(1, 11):
        r = oracle.keep_ratios(p, t, 1, 256, hbar[:, :t])
        if t < 7:
            assert r["t_star"][0] == 0 and r["act_scale"][0] == 0 and r["keep"][0] == 256
        else:
            assert r["t_star"][0] == int(gold["t_star"])
            assert r["act_scale"][0] == int(gold["act_scale"])
        if t == 7:
            assert r["keep"][0] == 256 and r["ratio_scale"][0] == 0.0   # t* itself is not pruned
        if t >= 8:
            assert abs(r["ratio_scale"][0] - float(gold[f"ratio_{t}"])) < 1e-12
            assert r["keep"][0] == int(gold[f"keep_{t}"])


def test_trigger_telescoping_and_linear_growth_never_triggers():
    p = oracle.SchedParams()
    # linear growth: smoothed rate equals eta forever, alpha < 1 -> never triggers
    hbar = (0.5 + 0.7 * np.arange(1, 14, dtype=np.float64))[None].astype(np.float32)
    r = oracle.keep_ratios(p, 13, 1, 100, hbar)
    assert r["t_star"][0] == 0 and r["keep"][0] == 100
    # telescoping: eta = (H_5 - H_1)/4 and smoothed g_t = (H_t - H_{t-2})/2, checked via the
    # trigger position on a random increasing-then-flat curve
    rng = np.random.default_rng(3)
    for _ in range(50):
        H = np.cumsum(rng.uniform(0.0, 1.0, 12))
        H[rng.integers(6, 12):] = H[5]
        eta = (H[4] - H[0]) / 4.0
        want = 0
        for t in range(6, 13):
            if (H[t - 1] - H[t - 3]) / 2.0 <= 0.5 * eta:
                want = t
                break
        # skip cases within fp32 rounding of the threshold
        margins = [abs((H[t - 1] - H[t - 3]) / 2.0 - 0.5 * eta) for t in range(6, 13)]
        if min(margins) < 1e-5:
            continue
        r = oracle.keep_ratios(p, 12, 1, 64, H[None].astype(np.float32))
        assert r["t_star"][0] == want


def test_scale_ratio_monotone_and_lambda_term():
    p0 = oracle.SchedParams(lam=0.0, force_act_scale=6)
    hbar = np.linspace(1, 3, 12, dtype=np.float32)[None]
    prev = -1.0
    for t in range(6, 13):
        r = oracle.keep_ratios(p0, t, 1, 1000, hbar[:, :t])["ratio_scale"][0]
        assert abs(r - 1.0 / (1.0 + math.exp(-(t - 6) / 0.8))) < 1e-12
        assert r > prev
        prev = r
    p1 = oracle.SchedParams(lam=0.1, force_act_scale=6)
    g = float(hbar[0, 7]) - float(hbar[0, 6])
    r = oracle.keep_ratios(p1, 8, 1, 1000, hbar[:, :8])["ratio_scale"][0]
    assert abs(r - (1.0 / (1.0 + math.exp(-2 / 0.8)) - 0.1 * math.tanh(g))) < 1e-12
    # growing entropy (g > 0) prunes less than a flat curve
    flat = np.full((1, 8), 2.0, np.float32)
    r_flat = oracle.keep_ratios(p1, 8, 1, 1000, flat)["ratio_scale"][0]
    assert r < r_flat


def test_layer_linkage_examples():
    p = oracle.SchedParams(force_act_scale=2, lam=0.0)
    hbar = np.array([[1.0, 1.0]], np.float32)          # t = 2 = activation -> Ratio_t = 0.5
    base = oracle.keep_ratios(p, 2, 1, 1000, hbar)
    assert base["ratio_scale"][0] == 0.5 and base["ratio_layer"][0] == 0.5
    same = oracle.keep_ratios(p, 2, 3, 1000, hbar, np.array([[4.0, 4.0, 4.0]], np.float32))
    assert same["ratio_layer"][0] == 0.5
    r2 = oracle.keep_ratios(p, 2, 2, 1000, hbar, np.array([[4.0, 5.0]], np.float32))
    assert abs(r2["ratio_layer"][0] - 0.75 * 0.5) < 1e-12      # Delta = 0.25
    assert r2["keep"][0] == 1000 - 375
    r3 = oracle.keep_ratios(p, 2, 3, 1000, hbar, np.array([[4.0, 5.0, 3.0]], np.float32))
    assert abs(r3["ratio_layer"][0] - (4.0 / 3.0) * 0.5) < 1e-12  # mu = 4.5, Delta = -1/3
    # a higher-entropy layer always prunes less
    assert r2["ratio_layer"][0] < 0.5 < r3["ratio_layer"][0]
    # mu == 0 -> Delta = 0
    rz = oracle.keep_ratios(p, 2, 2, 1000, hbar, np.array([[0.0, 5.0]], np.float32))
    assert rz["ratio_layer"][0] == 0.5


def test_keep_count_clamps_and_overrides():
    hbar = np.ones((2, 9), np.float32)
    p = oracle.SchedParams(force_act_scale=9, force_keep_ratio=0.2)
    r = oracle.keep_ratios(p, 9, 1, 16384, hbar)
    assert (r["keep"] == 16384 - math.floor(0.8 * 16384)).all() and r["keep"][0] == 3277
    p = oracle.SchedParams(force_act_scale=3, force_keep_ratio=0.0, k_min=5)
    assert oracle.keep_ratios(p, 9, 1, 100, hbar)["keep"][0] == 5
    p = oracle.SchedParams(force_act_scale=3, ratio_max=0.6, lam=0.0)
    assert oracle.keep_ratios(p, 9, 1, 100, hbar)["keep"][0] == 40      # sigmoid(7.5) clamped to 0.6
    # ratio driven above 1 or below 0 by the layer term is clamped
    p = oracle.SchedParams(force_act_scale=9, lam=0.0)
    hi = oracle.keep_ratios(p, 9, 2, 100, hbar, np.array([[4.0, 0.1], [1.0, 9.0]], np.float32))
    assert hi["ratio_layer"][0] > 0.9 and hi["keep"][0] == 100 - math.floor(hi["ratio_layer"][0] * 100)
    assert hi["ratio_layer"][1] < 0 and hi["keep"][1] == 100
    # not yet activated -> nothing pruned
    p = oracle.SchedParams(force_act_scale=10, force_keep_ratio=0.5)
    assert oracle.keep_ratios(p, 9, 1, 100, hbar)["keep"][0] == 100


# --------------------------------------------------------------------------- top-k
def _brute_topk(e, k):
    order = np.argsort(-e.astype(np.float64), kind="stable")   # descending, ties -> lower index
    keep = np.sort(order[:k])
    prune = np.sort(order[k:])
    return keep, prune


def test_topk_exhaustive_three_value_alphabet():
    alphabet = (0.0, 1.5, 1.5000001)
    for N in range(1, 8):
        rows = np.array(list(itertools.product(alphabet, repeat=N)), np.float32)
        for k in range(0, N + 1):
            ks = np.full(len(rows), k, np.int32)
            keep_idx, prune_idx, cu, pos = oracle.select_topk(rows, ks)
            assert np.array_equal(cu, np.arange(len(rows) + 1) * k)
            for s, e in enumerate(rows):
                wk, wp = _brute_topk(e, k)
                assert np.array_equal(keep_idx[s * k:(s + 1) * k], wk)
                assert np.array_equal(prune_idx[s * (N - k):(s + 1) * (N - k)], wp)
                inv = np.full(N, -1)
                inv[wk] = np.arange(k)
                assert np.array_equal(pos[s], inv)


def test_topk_special_cases_and_ragged_k():
    N = 97
    same = np.full((1, N), 2.5, np.float32)
    keep_idx, prune_idx, cu, _ = oracle.select_topk(same, [10])
    assert np.array_equal(keep_idx, np.arange(10)) and np.array_equal(prune_idx, np.arange(10, N))
    inc = np.arange(N, dtype=np.float32)[None]
    assert np.array_equal(oracle.select_topk(inc, [5])[0], np.arange(N - 5, N))
    assert np.array_equal(oracle.select_topk(inc, [N])[0], np.arange(N))
    e = np.array([[1, 7, 7, 3]], np.float32)
    assert oracle.select_topk(e, [1])[0][0] == 1            # first arg-max
    # signed zeros compare equal: the tie goes to the lower index
    z = np.array([[-0.0, 0.0, -0.0, 0.0]], np.float32)
    assert np.array_equal(oracle.select_topk(z, [2])[0], [0, 1])
    rng = np.random.default_rng(5)
    ent = rng.standard_normal((4, 300)).astype(np.float32)
    ent[:, ::7] = ent[:, 3:4]                                # many ties
    ks = np.array([1, 150, 299, 300], np.int32)
    keep_idx, prune_idx, cu, pos = oracle.select_topk(ent, ks)
    assert np.array_equal(cu, np.concatenate([[0], np.cumsum(ks)]))
    off_p = 0
    for s in range(4):
        wk, wp = _brute_topk(ent[s], ks[s])
        assert np.array_equal(keep_idx[cu[s]:cu[s + 1]], wk)
        assert np.array_equal(prune_idx[off_p:off_p + len(wp)], wp)
        off_p += len(wp)


# ------------------------------------------------------------------ block (Eq. 14)
def _rand_weights(C, F, rng, scale=0.2):
    w = {
        "ln1_g": 1 + 0.1 * rng.standard_normal(C), "ln1_b": 0.1 * rng.standard_normal(C),
        "w_qkv": scale * rng.standard_normal((3 * C, C)), "b_qkv": 0.1 * rng.standard_normal(3 * C),
        "w_o": scale * rng.standard_normal((C, C)), "b_o": 0.1 * rng.standard_normal(C),
        "ln2_g": 1 + 0.1 * rng.standard_normal(C), "ln2_b": 0.1 * rng.standard_normal(C),
        "w_fc1": scale * rng.standard_normal((F, C)), "b_fc1": 0.1 * rng.standard_normal(F),
        "w_fc2": scale * rng.standard_normal((C, F)), "b_fc2": 0.1 * rng.standard_normal(C),
    }
    return {k: v.astype(np.float32) for k, v in w.items()}


def _torch_block(w, eps, heads, x_kept, k_old, v_old):
    """One image, library ops only (torch fp64): x_kept [k, C], k_old/v_old [P, C]."""
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    x = t(x_kept)
    C = x.shape[1]
    dh = C // heads
    h = TF.layer_norm(x, (C,), t(w["ln1_g"]), t(w["ln1_b"]), eps)
    qkv = TF.linear(h, t(w["w_qkv"]), t(w["b_qkv"]))
    q, k, v = qkv.split(C, dim=1)
    K = torch.cat([t(k_old), k])
    Vv = torch.cat([t(v_old), v])
    sh = lambda a: a.view(a.shape[0], heads, dh).transpose(0, 1)
    o = TF.scaled_dot_product_attention(sh(q), sh(K), sh(Vv))
    o = o.transpose(0, 1).reshape(x.shape[0], C)
    x1 = x + TF.linear(o, t(w["w_o"]), t(w["b_o"]))
    h2 = TF.layer_norm(x1, (C,), t(w["ln2_g"]), t(w["ln2_b"]), eps)
    f = TF.linear(TF.gelu(TF.linear(h2, t(w["w_fc1"]), t(w["b_fc1"])), approximate="tanh"),
                  t(w["w_fc2"]), t(w["b_fc2"]))
    return (x1 + f).numpy(), k.numpy(), v.numpy()


def _block_case(seed=0, B=2, N=12, C=16, heads=2, F=24, Lmax=20, P=(5, 0)):
    rng = np.random.default_rng(seed)
    w = _rand_weights(C, F, rng)
    x = rng.standard_normal((B, N, C)).astype(np.float32)
    kc = rng.standard_normal((B, Lmax, C)).astype(np.float32)
    vc = rng.standard_normal((B, Lmax, C)).astype(np.float32)
    return w, x, kc, vc, np.array(P, np.int32)


def test_block_matches_library_composition_ragged():
    w, x, kc, vc, kv_len = _block_case()
    ent = np.random.default_rng(9).standard_normal((2, 12)).astype(np.float32)
    keep_idx, _, cu, _ = oracle.select_topk(ent, [7, 3])
    y, k_new, v_new = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len)
    for b in range(2):
        idx = keep_idx[cu[b]:cu[b + 1]]
        wy, wk, wv = _torch_block(w, 1e-6, 2, x[b, idx], kc[b, :kv_len[b]], vc[b, :kv_len[b]])
        assert np.allclose(y[cu[b]:cu[b + 1]], wy, atol=2e-5, rtol=1e-5)
        assert np.allclose(k_new[cu[b]:cu[b + 1]], wk, atol=1e-5)
        assert np.allclose(v_new[cu[b]:cu[b + 1]], wv, atol=1e-5)


def _torch_block_modulated(w, eps, heads, x_kept, k_old, v_old, md):
    """The adaptive-LayerNorm block of one image from library ops (torch fp64): md holds the
    image's six [C] vectors."""
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    x = t(x_kept)
    C = x.shape[1]
    dh = C // heads
    h = TF.layer_norm(x, (C,), t(w["ln1_g"]), t(w["ln1_b"]), eps) * (1 + t(md["scale1"])) + t(md["shift1"])
    q, k, v = TF.linear(h, t(w["w_qkv"]), t(w["b_qkv"])).split(C, dim=1)
    K, Vv = torch.cat([t(k_old), k]), torch.cat([t(v_old), v])
    sh = lambda a: a.view(a.shape[0], heads, dh).transpose(0, 1)
    o = TF.scaled_dot_product_attention(sh(q), sh(K), sh(Vv)).transpose(0, 1).reshape(x.shape[0], C)
    x1 = x + t(md["gate1"]) * TF.linear(o, t(w["w_o"]), t(w["b_o"]))
    h2 = TF.layer_norm(x1, (C,), t(w["ln2_g"]), t(w["ln2_b"]), eps) * (1 + t(md["scale2"])) + t(md["shift2"])
    f = TF.linear(TF.gelu(TF.linear(h2, t(w["w_fc1"]), t(w["b_fc1"])), approximate="tanh"),
                  t(w["w_fc2"]), t(w["b_fc2"]))
    return (x1 + t(md["gate2"]) * f).numpy(), k.numpy(), v.numpy()


def _rand_modulation(B, C, rng):
    return {n: (0.5 * rng.standard_normal((B, C))).astype(np.float32) for n in oracle.MODULATION_NAMES}


def test_modulated_block_matches_library_composition():
    """Adaptive LayerNorm (per-image scale/shift after each LayerNorm, per-image gate on each branch)
    against the same block composed from library ops per image, ragged keep counts."""
    w, x, kc, vc, kv_len = _block_case(seed=4)
    md = _rand_modulation(2, 16, np.random.default_rng(40))
    ent = np.random.default_rng(9).standard_normal((2, 12)).astype(np.float32)
    keep_idx, _, cu, _ = oracle.select_topk(ent, [7, 3])
    y, k_new, v_new = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len, modulation=md)
    for b in range(2):
        idx = keep_idx[cu[b]:cu[b + 1]]
        mb = {n: a[b] for n, a in md.items()}
        wy, wk, wv = _torch_block_modulated(w, 1e-6, 2, x[b, idx], kc[b, :kv_len[b]], vc[b, :kv_len[b]], mb)
        assert np.allclose(y[cu[b]:cu[b + 1]], wy, atol=2e-5, rtol=1e-5)
        assert np.allclose(k_new[cu[b]:cu[b + 1]], wk, atol=1e-5)
        assert np.allclose(v_new[cu[b]:cu[b + 1]], wv, atol=1e-5)


def test_modulated_block_special_cases():
    """What the modulation terms must reduce to: no scale, no shift, unit gates = the plain block,
    bit for bit; both gates 0 = the identity on the kept rows whatever the rest holds; gate2 = 0 leaves
    the attention half only, which does not depend on the second LayerNorm's modulation; a missing
    entry means no such term."""
    w, x, kc, vc, kv_len = _block_case(seed=6)
    B, N, C = x.shape
    ent = np.random.default_rng(3).standard_normal((B, N)).astype(np.float32)
    keep_idx, _, cu, _ = oracle.select_topk(ent, [5, 9])
    plain, pk, pv = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len)
    zeros, ones = np.zeros((B, C), np.float32), np.ones((B, C), np.float32)
    ident = dict(shift1=zeros, scale1=zeros, gate1=ones, shift2=zeros, scale2=zeros, gate2=ones)
    y, k_new, v_new = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len, modulation=ident)
    assert np.array_equal(y, plain) and np.array_equal(k_new, pk) and np.array_equal(v_new, pv)
    y, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len, modulation={})
    assert np.array_equal(y, plain)
    md = _rand_modulation(B, C, np.random.default_rng(41))
    md["gate1"], md["gate2"] = zeros, zeros
    y, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len, modulation=md)
    xk = np.concatenate([x[b, keep_idx[cu[b]:cu[b + 1]]] for b in range(B)])
    assert np.array_equal(y, xk)
    md = _rand_modulation(B, C, np.random.default_rng(42))
    md["gate2"] = zeros
    ya, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len, modulation=md)
    md2 = dict(md, scale2=md["scale2"] + 3, shift2=md["shift2"] - 2)
    yb, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len, modulation=md2)
    assert np.array_equal(ya, yb)
    assert not np.allclose(ya, plain, atol=1e-3)


def test_block_keep_all_equals_dense_block_and_row_subset():
    w, x, kc, vc, kv_len = _block_case(seed=2)
    B, N, _ = x.shape
    keep_idx = np.tile(np.arange(N, dtype=np.int32), B)
    cu = np.arange(B + 1, dtype=np.int32) * N
    y, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len)
    for b in range(B):
        wy, _, _ = _torch_block(w, 1e-6, 2, x[b], kc[b, :kv_len[b]], vc[b, :kv_len[b]])
        assert np.allclose(y[b * N:(b + 1) * N], wy, atol=2e-5, rtol=1e-5)
    rows = np.array([3, 17, 0], np.int32)
    ys, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len, rows=rows)
    assert np.array_equal(ys, y[rows])


def test_block_attention_special_cases():
    w, x, kc, vc, kv_len = _block_case(seed=3, P=(4, 6))
    B, N, C = x.shape
    # isolate attention: q = 0 -> uniform weights; W_o = I, FFN output zero, k/v = LN1 output
    w["w_qkv"][:C] = 0
    w["b_qkv"][:C] = 0
    w["w_qkv"][2 * C:] = np.eye(C, dtype=np.float32)
    w["b_qkv"][2 * C:] = 0
    w["w_o"] = np.eye(C, dtype=np.float32)
    w["b_o"][:] = 0
    w["w_fc2"][:] = 0
    w["b_fc2"][:] = 0
    keep_idx = np.array([1, 4, 9, 0, 2], np.int32)
    cu = np.array([0, 3, 5], np.int32)
    y, k_new, v_new = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len)
    for b in range(B):
        allv = np.concatenate([vc[b, :kv_len[b]], v_new[cu[b]:cu[b + 1]]]).astype(np.float64)
        for m in range(cu[b], cu[b + 1]):
            assert np.allclose(y[m] - x[b, keep_idx[m]], allv.mean(axis=0), atol=1e-5)
    # one key only (empty cache, one kept token): the output is that token's own value row
    y1, _, v1 = oracle.pruned_block_forward(w, 1e-6, 2, x, np.array([5, 7], np.int32),
                                            np.array([0, 1, 2], np.int32), kc, vc,
                                            np.zeros(2, np.int32))
    assert np.allclose(y1[0] - x[0, 5], v1[0], atol=1e-6)
    assert np.allclose(y1[1] - x[1, 7], v1[1], atol=1e-6)


def test_block_constant_query_softmax_per_head():
    from scipy.special import softmax
    w, x, kc, vc, kv_len = _block_case(seed=4, B=1, P=(9,))
    C, heads, dh = 16, 2, 8
    w["w_qkv"][:C] = 0                      # q = b_q for every token
    w["w_o"] = np.eye(C, dtype=np.float32)
    w["b_o"][:] = 0
    w["w_fc2"][:] = 0
    w["b_fc2"][:] = 0
    keep_idx = np.array([2, 3], np.int32)
    cu = np.array([0, 2], np.int32)
    y, k_new, v_new = oracle.pruned_block_forward(w, 1e-6, heads, x, keep_idx, cu, kc, vc, kv_len)
    K = np.concatenate([kc[0, :9], k_new]).astype(np.float64)
    Vv = np.concatenate([vc[0, :9], v_new]).astype(np.float64)
    q = w["b_qkv"][:C].astype(np.float64)
    want = np.zeros(C)
    for hd in range(heads):
        sl = slice(hd * dh, (hd + 1) * dh)
        pr = softmax(K[:, sl] @ q[sl] / math.sqrt(dh))
        want[sl] = pr @ Vv[:, sl]
    for m in range(2):
        assert np.allclose(y[m] - x[0, keep_idx[m]], want, atol=1e-5)


def test_block_layernorm_and_linear_probes():
    w, x, kc, vc, kv_len = _block_case(seed=5, B=1, P=(0,))
    C = 16
    w["w_qkv"][C:2 * C] = np.eye(C, dtype=np.float32)   # k_new = LN1(x)
    w["b_qkv"][C:2 * C] = 0
    x[0, 0] = 3.25                                       # constant row -> LN gives beta
    x[0, 2] = 7.0 * x[0, 1]                              # positive scaling leaves LN unchanged
    keep_idx = np.arange(6, dtype=np.int32)
    cu = np.array([0, 6], np.int32)
    _, k_new, v_new = oracle.pruned_block_forward(w, 1e-12, 2, x, keep_idx, cu, kc, vc, kv_len)
    assert np.allclose(k_new[0], w["ln1_b"], atol=1e-6)
    assert np.allclose(k_new[1], k_new[2], atol=1e-5)
    unit = (k_new[3].astype(np.float64) - w["ln1_b"]) / w["ln1_g"]
    assert abs(unit.mean()) < 1e-6 and abs(unit.var() - 1.0) < 1e-5
    # v_new = LN1(x) W_v^T + b_v with [out, in] weights: check with a numpy matmul
    want_v = k_new.astype(np.float64) @ w["w_qkv"][2 * C:].astype(np.float64).T + w["b_qkv"][2 * C:]
    assert np.allclose(v_new, want_v, atol=1e-5)


def test_block_ffn_path_against_library():
    w, x, kc, vc, kv_len = _block_case(seed=6, B=1, P=(3,))
    C = 16
    w["w_o"][:] = 0
    w["b_o"][:] = 0                                      # x1 = x
    keep_idx = np.array([0, 5, 6, 11], np.int32)
    cu = np.array([0, 4], np.int32)
    y, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len)
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    xs = t(x[0, keep_idx])
    h2 = TF.layer_norm(xs, (C,), t(w["ln2_g"]), t(w["ln2_b"]), 1e-6)
    f = TF.linear(TF.gelu(TF.linear(h2, t(w["w_fc1"]), t(w["b_fc1"])), approximate="tanh"),
                  t(w["w_fc2"]), t(w["b_fc2"]))
    assert np.allclose(y, (xs + f).numpy(), atol=1e-5)


def test_block_kept_set_permutation_equivariance():
    # permuting the tokens of x_in together with keep_idx leaves every kept row's output unchanged
    w, x, kc, vc, kv_len = _block_case(seed=7, B=1, P=(5,))
    keep_idx = np.array([1, 3, 8, 10], np.int32)
    cu = np.array([0, 4], np.int32)
    y, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len)
    perm = np.random.default_rng(0).permutation(12)
    inv = np.argsort(perm)
    x_p = x[:, perm]
    keep_p = inv[keep_idx].astype(np.int32)              # same tokens, new positions, same order
    y_p, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x_p, keep_p, cu, kc, vc, kv_len)
    assert np.allclose(y, y_p, atol=1e-6)


# ---------------------------------------------------------------- restore (Eq. 15-16)
def _restore_case(seed, B, hp, wp, h, w, C, k):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((B, h * w, C)).astype(np.float32)
    cache = rng.standard_normal((B, hp, wp, C)).astype(np.float32)
    ent = rng.standard_normal((B, h * w)).astype(np.float32)
    keep_idx, prune_idx, cu, _ = oracle.select_topk(ent, k)
    y = rng.standard_normal((int(cu[-1]), C)).astype(np.float32)
    return x, cache, keep_idx, prune_idx, cu, y


def test_restore_matches_library_bilinear_and_cache_definition():
    B, hp, wp, h, w, C = 2, 5, 5, 8, 8, 6
    x, cache, keep_idx, prune_idx, cu, y = _restore_case(0, B, hp, wp, h, w, C, [20, 33])
    x_out, cache_out = oracle.restore_from_cache(x, y, keep_idx, prune_idx, cu, cache, h, w)
    up = TF.interpolate(torch.from_numpy(cache.astype(np.float64)).permute(0, 3, 1, 2), size=(h, w),
                        mode="bilinear", align_corners=False).permute(0, 2, 3, 1).reshape(B, h * w, C).numpy()
    off = 0
    for b in range(B):
        kept = keep_idx[cu[b]:cu[b + 1]]
        npr = h * w - len(kept)
        pruned = prune_idx[off:off + npr]
        off += npr
        assert np.array_equal(x_out[b, kept], y[cu[b]:cu[b + 1]])          # kept rows bit-equal y
        assert np.allclose(cache_out[b, kept], y[cu[b]:cu[b + 1]] - x[b, kept], atol=1e-6)
        assert np.allclose(x_out[b, pruned], x[b, pruned] + up[b, pruned], atol=1e-5)
        assert np.allclose(cache_out[b, pruned], up[b, pruned], atol=1e-6)
        assert np.allclose(x_out[b] - x[b], cache_out[b], atol=1e-5)        # Eq. 15 on every row


def test_restore_non_square_and_downscale_factor_library():
    B, hp, wp, h, w, C = 1, 13, 13, 16, 16, 3
    x, cache, keep_idx, prune_idx, cu, y = _restore_case(1, B, hp, wp, h, w, C, [0])
    x_out, cache_out = oracle.restore_from_cache(x, y, keep_idx, prune_idx, cu, cache, h, w)
    up = TF.interpolate(torch.from_numpy(cache.astype(np.float64)).permute(0, 3, 1, 2), size=(h, w),
                        mode="bilinear", align_corners=False).permute(0, 2, 3, 1).reshape(B, h * w, C).numpy()
    assert np.allclose(cache_out, up, atol=1e-6)
    # rectangular source grid
    rng = np.random.default_rng(2)
    cache = rng.standard_normal((1, 3, 7, 2)).astype(np.float32)
    x = np.zeros((1, 6 * 9, 2), np.float32)
    pr = np.arange(54, dtype=np.int32)
    _, co = oracle.restore_from_cache(x, np.zeros((0, 2), np.float32), np.zeros(0, np.int32), pr,
                                      np.array([0, 0], np.int32), cache, 6, 9)
    up = TF.interpolate(torch.from_numpy(cache.astype(np.float64)).permute(0, 3, 1, 2), size=(6, 9),
                        mode="bilinear", align_corners=False).permute(0, 2, 3, 1).reshape(1, 54, 2).numpy()
    assert np.allclose(co, up, atol=1e-6)


def test_restore_closed_forms():
    z0 = np.zeros(0, np.int32)
    cu0 = np.array([0, 0], np.int32)
    # 1-D 2 -> 4: (a, .75a+.25b, .25a+.75b, b)
    a, b = 2.0, 10.0
    cache = np.array([a, b], np.float32).reshape(1, 1, 2, 1)
    x = np.zeros((1, 4, 1), np.float32)
    _, co = oracle.restore_from_cache(x, np.zeros((0, 1), np.float32), z0, np.arange(4, dtype=np.int32),
                                      cu0, cache, 1, 4)
    assert np.allclose(co.ravel(), [a, .75 * a + .25 * b, .25 * a + .75 * b, b], atol=1e-6)
    # same size -> identity; constant -> constant; 1x1 -> broadcast
    rng = np.random.default_rng(3)
    cache = rng.standard_normal((1, 4, 4, 2)).astype(np.float32)
    x = rng.standard_normal((1, 16, 2)).astype(np.float32)
    xo, co = oracle.restore_from_cache(x, np.zeros((0, 2), np.float32), z0, np.arange(16, dtype=np.int32),
                                       cu0, cache, 4, 4)
    assert np.array_equal(co, cache.reshape(1, 16, 2))
    assert np.allclose(xo, x + cache.reshape(1, 16, 2), atol=1e-6)
    const = np.full((1, 3, 3, 2), 1.75, np.float32)
    _, co = oracle.restore_from_cache(x, np.zeros((0, 2), np.float32), z0, np.arange(16, dtype=np.int32),
                                      cu0, const, 4, 4)
    assert np.allclose(co, 1.75, atol=1e-7)
    one = rng.standard_normal((1, 1, 1, 2)).astype(np.float32)
    _, co = oracle.restore_from_cache(x, np.zeros((0, 2), np.float32), z0, np.arange(16, dtype=np.int32),
                                      cu0, one, 4, 4)
    assert np.allclose(co, np.broadcast_to(one.reshape(1, 1, 2), (1, 16, 2)), atol=1e-7)
    # zero cache -> pruned rows pass through unchanged
    xo, _ = oracle.restore_from_cache(x, np.zeros((0, 2), np.float32), z0, np.arange(16, dtype=np.int32),
                                      cu0, np.zeros((1, 2, 2, 2), np.float32), 4, 4)
    assert np.array_equal(xo, x)


# ------------------------------------------------------------------- whole step
def test_whole_step_keep_all_reproduces_dense_layer():
    w, x, kc, vc, kv_len = _block_case(seed=8, B=2, N=16, P=(5, 2))
    B, N, C = x.shape
    ent, _ = oracle.scale_entropy(np.random.default_rng(0).standard_normal((B, N, 32)).astype(np.float32))
    r = oracle.keep_ratios(oracle.SchedParams(), 3, 1, N, np.ones((B, 3), np.float32))
    assert (r["keep"] == N).all()                       # before t_est nothing is pruned
    keep_idx, prune_idx, cu, _ = oracle.select_topk(ent, r["keep"])
    assert len(prune_idx) == 0
    y, _, _ = oracle.pruned_block_forward(w, 1e-6, 2, x, keep_idx, cu, kc, vc, kv_len)
    cache = np.random.default_rng(1).standard_normal((B, 3, 3, C)).astype(np.float32)
    x_out, cache_out = oracle.restore_from_cache(x, y, keep_idx, prune_idx, cu, cache, 4, 4)
    for b in range(B):
        wy, _, _ = _torch_block(w, 1e-6, 2, x[b], kc[b, :kv_len[b]], vc[b, :kv_len[b]])
        assert np.allclose(x_out[b], wy, atol=2e-5, rtol=1e-5)
        assert np.allclose(cache_out[b], wy - x[b], atol=3e-5)


# ------------------------------------------------------------------ alternative selection scores
def test_score_mse_pins():
    """Closed forms and a library composition: same-size reference -> plain mean squared difference;
    constant reference -> mean (x - const)^2; torch's bilinear interpolation (fp64) for a real resize;
    a token equal to the resized reference scores 0."""
    import torch.nn.functional as F
    rng = np.random.default_rng(0)
    B, h, w, C = 2, 6, 9, 16
    x = rng.standard_normal((B, h * w, C)).astype(np.float32)
    same = rng.standard_normal((B, h, w, C)).astype(np.float32)
    got = oracle.score_mse(x, same, h, w)
    assert np.allclose(got, ((x - same.reshape(B, h * w, C)).astype(np.float64) ** 2).mean(-1), rtol=1e-6)
    const = np.full((B, 3, 4, C), 0.75, np.float32)
    assert np.allclose(oracle.score_mse(x, const, h, w), ((x.astype(np.float64) - 0.75) ** 2).mean(-1), rtol=1e-6)
    ref = rng.standard_normal((B, 4, 5, C)).astype(np.float32)
    up = F.interpolate(torch.from_numpy(ref).double().permute(0, 3, 1, 2), size=(h, w), mode="bilinear",
                       align_corners=False).permute(0, 2, 3, 1).reshape(B, h * w, C).numpy()
    assert np.allclose(oracle.score_mse(x, ref, h, w), ((x - up) ** 2).mean(-1), rtol=1e-5)
    assert np.abs(oracle.score_mse(up.astype(np.float32), ref, h, w)).max() < 1e-12
    # a token moved away from the prediction scores higher: the criterion ranks by detail energy
    x2 = up.astype(np.float32).copy()
    x2[0, 7] += 0.5
    s = oracle.score_mse(x2, ref, h, w)
    assert s[0].argmax() == 7 and abs(s[0, 7] - 0.25) < 1e-6


def test_score_attention_mass_pins():
    """Zero queries -> every key gets 1 / (prior + N) of every row; the scores of an image sum to the
    share of attention that stays inside the scale (1 without prior keys); a key every query is
    aligned with collects almost everything; torch softmax (fp64) on random inputs with ragged prior
    lengths; per-head layout (head h uses channels [h*dh, (h+1)*dh))."""
    rng = np.random.default_rng(1)
    B, N, heads, dh, Lmax = 2, 12, 3, 8, 20
    C = heads * dh
    q = rng.standard_normal((B, N, C)).astype(np.float32)
    k = rng.standard_normal((B, N, C)).astype(np.float32)
    kc = rng.standard_normal((B, Lmax, C)).astype(np.float32)
    lens = np.array([7, 0], np.int32)
    got = oracle.score_attention_mass(np.zeros_like(q), k, kc, lens, heads)
    assert np.allclose(got[0], 1.0 / (7 + N)) and np.allclose(got[1], 1.0 / N)
    got = oracle.score_attention_mass(q, k, kc, lens, heads)
    want = np.zeros((B, N))
    for b in range(B):
        keys = np.concatenate([kc[b, :lens[b]], k[b]], 0).astype(np.float64)
        for hd in range(heads):
            sl = slice(hd * dh, (hd + 1) * dh)
            p = torch.softmax(torch.from_numpy(q[b, :, sl].astype(np.float64) @ keys[:, sl].T / np.sqrt(dh)), dim=-1).numpy()
            want[b] += p[:, lens[b]:].sum(0)
    want /= heads * N
    assert np.allclose(got, want, rtol=1e-6, atol=1e-9)
    assert abs(got[1].sum() - 1.0) < 1e-6 and got[0].sum() < 1.0
    # one key aligned with every query in every head
    q2 = np.tile(rng.standard_normal((1, 1, C)).astype(np.float32), (1, N, 1)) * 3
    k2 = 0.01 * rng.standard_normal((1, N, C)).astype(np.float32)
    k2[0, 5] = q2[0, 0] * 3
    s = oracle.score_attention_mass(q2, k2, None, None, heads)
    assert s[0].argmax() == 5 and s[0, 5] > 0.99
    # swapping two heads' channel blocks in q and k alike leaves the scores unchanged
    perm = np.r_[np.arange(dh, 2 * dh), np.arange(0, dh), np.arange(2 * dh, C)]
    assert np.allclose(oracle.score_attention_mass(q[..., perm], k[..., perm], kc[..., perm], lens, heads), got, rtol=1e-6)


# ------------------------------------------------- block variants: rotary embedding, QK norm, cross-attention
def _ext_case(rng, B=2, N=10, heads=2, dh=8, F=24, Lmax=14, Lc=5):
    C = heads * dh
    names = {"ln1_g": (C,), "ln1_b": (C,), "w_qkv": (3 * C, C), "b_qkv": (3 * C,), "w_o": (C, C), "b_o": (C,),
             "ln2_g": (C,), "ln2_b": (C,), "w_fc1": (F, C), "b_fc1": (F,), "w_fc2": (C, F), "b_fc2": (C,)}
    w = {n: (0.3 * rng.standard_normal(sh)).astype(np.float32) for n, sh in names.items()}
    w["ln1_g"] += 1
    w["ln2_g"] += 1
    x = rng.standard_normal((B, N, C)).astype(np.float32)
    kc = rng.standard_normal((B, Lmax, C)).astype(np.float32)
    vc = rng.standard_normal((B, Lmax, C)).astype(np.float32)
    lens = np.array([4, 0], np.int32)[:B]
    keep = [np.sort(rng.choice(N, size=k, replace=False)).astype(np.int32) for k in (7, 3)[:B]]
    keep_idx = np.concatenate(keep)
    cu = np.r_[0, np.cumsum([len(k) for k in keep])].astype(np.int32)
    ang = rng.uniform(0, 2 * np.pi, (N, dh // 2))
    ext = dict(rope_cos=np.cos(ang).astype(np.float32), rope_sin=np.sin(ang).astype(np.float32),
               qk_gain_q=(1 + 0.2 * rng.standard_normal(C)).astype(np.float32),
               qk_gain_k=(1 + 0.2 * rng.standard_normal(C)).astype(np.float32),
               lnc_g=(1 + 0.1 * rng.standard_normal(C)).astype(np.float32), lnc_b=(0.1 * rng.standard_normal(C)).astype(np.float32),
               w_q2=(0.3 * rng.standard_normal((C, C))).astype(np.float32), b_q2=(0.1 * rng.standard_normal(C)).astype(np.float32),
               w_o2=(0.3 * rng.standard_normal((C, C))).astype(np.float32), b_o2=(0.1 * rng.standard_normal(C)).astype(np.float32),
               ck=rng.standard_normal((B, Lc, C)).astype(np.float32), cv=rng.standard_normal((B, Lc, C)).astype(np.float32),
               cond_len=np.array([Lc, 2], np.int32)[:B])
    return dict(w=w, x=x, kc=kc, vc=vc, lens=lens, keep_idx=keep_idx, cu=cu, heads=heads, dh=dh, C=C, F=F, ext=ext, N=N, B=B)


def _ext_torch(c, ext):
    """The extended block as a composition of torch library ops in float64 (independent of the
    oracle's loops): F.layer_norm, F.linear, F.normalize, complex multiplication for the rotation,
    F.scaled_dot_product_attention, F.gelu(tanh)."""
    import torch.nn.functional as Fn
    t = lambda a: torch.from_numpy(np.asarray(a)).double()
    w = {n: t(v) for n, v in c["w"].items()}
    heads, dh, C, B = c["heads"], c["dh"], c["C"], c["B"]
    ys, ks = [], []

    def transform(v, gain, pos):                       # v [n, C]
        v = v.view(-1, heads, dh)
        if gain is not None:
            v = Fn.normalize(v, dim=-1, eps=1e-12) * t(gain).view(heads, dh)
        if ext.get("rope_cos") is not None:
            rot = torch.complex(t(ext["rope_cos"])[pos], t(ext["rope_sin"])[pos]).unsqueeze(1)        # [n, 1, dh/2]
            v = torch.view_as_real(torch.view_as_complex(v.reshape(-1, heads, dh // 2, 2).contiguous()) * rot).reshape(-1, heads, dh)
        return v.reshape(-1, C)

    for b in range(B):
        idx = c["keep_idx"][c["cu"][b]:c["cu"][b + 1]]
        xb = t(c["x"][b, idx])
        h = Fn.layer_norm(xb, (C,), w["ln1_g"], w["ln1_b"], 1e-6)
        qkv = Fn.linear(h, w["w_qkv"], w["b_qkv"])
        q, k, v = qkv[:, :C], qkv[:, C:2 * C], qkv[:, 2 * C:]
        q = transform(q.contiguous(), ext.get("qk_gain_q"), idx)
        k = transform(k.contiguous(), ext.get("qk_gain_k"), idx)
        n0 = c["lens"][b]
        K = torch.cat([t(c["kc"][b, :n0]), k], 0).view(-1, heads, dh).transpose(0, 1)
        V = torch.cat([t(c["vc"][b, :n0]), v], 0).view(-1, heads, dh).transpose(0, 1)
        o = Fn.scaled_dot_product_attention(q.view(-1, heads, dh).transpose(0, 1), K, V).transpose(0, 1).reshape(-1, C)
        x1 = xb + Fn.linear(o, w["w_o"], w["b_o"])
        if ext.get("w_q2") is not None:
            hc = Fn.layer_norm(x1, (C,), t(ext["lnc_g"]), t(ext["lnc_b"]), 1e-6)
            q2 = Fn.linear(hc, t(ext["w_q2"]), t(ext["b_q2"])).view(-1, heads, dh).transpose(0, 1)
            n_c = int(ext["cond_len"][b])
            Kc = t(ext["ck"][b, :n_c]).view(-1, heads, dh).transpose(0, 1)
            Vc = t(ext["cv"][b, :n_c]).view(-1, heads, dh).transpose(0, 1)
            o2 = Fn.scaled_dot_product_attention(q2, Kc, Vc).transpose(0, 1).reshape(-1, C)
            x1 = x1 + Fn.linear(o2, t(ext["w_o2"]), t(ext["b_o2"]))
        h2 = Fn.layer_norm(x1, (C,), w["ln2_g"], w["ln2_b"], 1e-6)
        ys.append(x1 + Fn.linear(Fn.gelu(Fn.linear(h2, w["w_fc1"], w["b_fc1"]), approximate="tanh"), w["w_fc2"], w["b_fc2"]))
        ks.append(k)
    return torch.cat(ys).numpy(), torch.cat(ks).numpy()


def _run_ext(c, ext, **kw):
    return oracle.pruned_block_forward_ext(c["w"], 1e-6, c["heads"], c["x"], c["keep_idx"], c["cu"], c["kc"], c["vc"],
                                           c["lens"], ext, **kw)


def test_block_ext_matches_library_composition():
    rng = np.random.default_rng(5)
    c = _ext_case(rng)
    full = c["ext"]
    subsets = [full,
               {k: full[k] for k in ("rope_cos", "rope_sin")},
               {k: full[k] for k in ("qk_gain_q", "qk_gain_k")},
               {k: full[k] for k in ("lnc_g", "lnc_b", "w_q2", "b_q2", "w_o2", "b_o2", "ck", "cv", "cond_len")}]
    for ext in subsets:
        y, k_new, _ = _run_ext(c, ext)
        wy, wk = _ext_torch(c, ext)
        assert np.abs(y - wy).max() < 2e-5 and np.abs(k_new - wk).max() < 2e-5


def test_block_ext_reductions_and_invariants():
    rng = np.random.default_rng(6)
    c = _ext_case(rng)
    full = c["ext"]
    plain, k_plain, _ = oracle.pruned_block_forward(c["w"], 1e-6, c["heads"], c["x"], c["keep_idx"], c["cu"], c["kc"],
                                                    c["vc"], c["lens"])
    # nothing switched on, and the identity rotation: the plain block, bit for bit
    y, k_new, _ = _run_ext(c, {})
    assert np.array_equal(y, plain) and np.array_equal(k_new, k_plain)
    ident = dict(rope_cos=np.ones_like(full["rope_cos"]), rope_sin=np.zeros_like(full["rope_sin"]))
    assert np.array_equal(_run_ext(c, ident)[0], plain)
    # rotation: with no prior keys, turning every position by the same extra angle changes nothing
    # (scores depend on angle differences only), while the rotated keys themselves do change
    c0 = dict(c, lens=np.zeros_like(c["lens"]))
    ang = np.arctan2(full["rope_sin"], full["rope_cos"])
    a = dict(rope_cos=np.cos(ang).astype(np.float32), rope_sin=np.sin(ang).astype(np.float32))
    b = dict(rope_cos=np.cos(ang + 0.7).astype(np.float32), rope_sin=np.sin(ang + 0.7).astype(np.float32))
    ya, ka, _ = _run_ext(c0, a)
    yb, kb, _ = _run_ext(c0, b)
    assert np.abs(ya - yb).max() < 1e-5 and np.abs(ka - kb).max() > 0.1
    assert np.abs(ya - _run_ext(c0, {})[0]).max() > 1e-3                 # and the rotation does act
    # QK normalisation: the scale of a head's query projection no longer matters
    qk = {k: full[k] for k in ("qk_gain_q", "qk_gain_k")}
    w2 = dict(c["w"])
    w2["w_qkv"] = c["w"]["w_qkv"].copy()
    w2["b_qkv"] = c["w"]["b_qkv"].copy()
    w2["w_qkv"][: c["dh"]] *= 3.0
    w2["b_qkv"][: c["dh"]] *= 3.0
    y1 = _run_ext(c, qk)[0]
    y2 = _run_ext(dict(c, w=w2), qk)[0]
    assert np.abs(y1 - y2).max() < 1e-5
    assert np.abs(_run_ext(dict(c, w=w2), {})[0] - plain).max() > 1e-3   # without it, it does
    # unit keys: every transformed key head has norm |gain| when the gain is constant
    g1 = dict(qk_gain_q=np.full(c["C"], 2.0, np.float32), qk_gain_k=np.full(c["C"], 0.5, np.float32))
    kn = _run_ext(c, g1)[1].reshape(-1, c["heads"], c["dh"])
    assert np.allclose(np.linalg.norm(kn, axis=-1), 0.5, atol=1e-6)
    # cross-attention: a zero output projection leaves the plain block; one condition token adds
    # exactly its projected value row to the residual stream before the MLP
    cross = {k: full[k] for k in ("lnc_g", "lnc_b", "w_q2", "b_q2", "w_o2", "b_o2", "ck", "cv", "cond_len")}
    z = dict(cross, w_o2=np.zeros_like(cross["w_o2"]), b_o2=np.zeros_like(cross["b_o2"]))
    assert np.array_equal(_run_ext(c, z)[0], plain)
    one = dict(cross, cond_len=np.ones(c["B"], np.int32))
    wz = dict(c["w"], w_fc2=np.zeros_like(c["w"]["w_fc2"]), b_fc2=np.zeros_like(c["w"]["b_fc2"]))   # y = x1
    y_one = _run_ext(dict(c, w=wz), one)[0]
    y_base = oracle.pruned_block_forward(wz, 1e-6, c["heads"], c["x"], c["keep_idx"], c["cu"], c["kc"], c["vc"], c["lens"])[0]
    for b_ in range(c["B"]):
        add = cross["w_o2"].astype(np.float64) @ cross["cv"][b_, 0].astype(np.float64) + cross["b_o2"]
        rows = slice(c["cu"][b_], c["cu"][b_ + 1])
        assert np.abs((y_one[rows] - y_base[rows]) - add).max() < 1e-5
    # row subsets evaluate to the same rows
    sub = np.array([0, 3, 8], np.int32)
    assert np.array_equal(_run_ext(c, full, rows=sub)[0], _run_ext(c, full)[0][sub])

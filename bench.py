#!/usr/bin/env python
"""Benchmark of the NOVA pruned-scale step on B200.

A step is one pass of the whole hot path over one accelerated scale: for each of the L layers,
entropy of that layer's logits -> keep counts (host) -> top-k -> block on the kept tokens ->
restore from the residual cache. The default workload is the 1024x1024 large-model shape
(32 layers, width 2048, 16 heads x 128, MLP 8192, last scale 64x64 = 4096 tokens attending to
6425 prior tokens, batch 4, keep ratio 0.5). Prints one JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import nova_synth as synth  # noqa: E402

METRIC = "pruned_scale_images_per_s"
UNIT = "images/s"
NOMINAL_PEAKS = {"hbm": 8000.0, "tensor": 2250.0}      # GB/s, dense bf16 TFLOP/s (context; `peak` is the measured one)
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic_c4_1024_batch4_keep0.5.txt")


def source_digest(paths):
    import hashlib
    h = hashlib.sha256()
    for p in paths:
        with open(os.path.join(ROOT, p), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic():
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the committed ncu capture
    on the default workload's launch shapes, per kernel key. Each line of the summary file names the
    sources the kernel is built from and their digest at capture time: a kernel whose sources have
    changed since reports no traffic (None) until it is captured again."""
    out = {}
    try:
        for line in open(TRAFFIC_FILE):
            f = line.split()
            if len(f) < 4 or line.startswith("#"):
                continue
            key, nbytes, digest, srcs = f[0], int(f[1]), f[2], f[3].split(",")
            out[key] = nbytes if source_digest(srcs) == digest else None
    except (OSError, ValueError):
        pass
    return out


CONTRACTIONS = ("attention", "gemm_qkv", "gemm_proj", "gemm_fc1", "gemm_fc2")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4_1024", choices=sorted(synth.CONFIGS))
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--keep", type=float, default=0.5)
    ap.add_argument("--scale", type=int, default=None, help="1-based scale index (default: last)")
    ap.add_argument("--layers", type=int, default=None, help="override the number of layers (small profiling cases)")
    ap.add_argument("--two-call-layers", action="store_true",
                    help="time nova_pruned_block_forward + nova_restore_from_cache per layer instead of the one "
                         "nova_pruned_layer_forward call (the other form is timed after the timed region either way)")
    ap.add_argument("--all-configs", action="store_true",
                    help="one JSON line per stated configuration (the five workloads; the 1024 shape at keep ratios "
                         "0.25 / 0.5 / 0.75 and batch 1 / 4), device-resident timing only")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-next", action="store_true",
                    help="skip the extra timings after the timed region (fused head entropy, device-driven step)")
    return ap.parse_args()


def workload_desc(args):
    ms = synth.CONFIGS[args.workload]
    if args.layers:
        import dataclasses
        ms = dataclasses.replace(ms, L=args.layers, name=f"{ms.name}[{args.layers} layers]")
    t = args.scale or len(ms.scales)
    B = args.batch or ms.B
    side = ms.scales[t - 1]
    prev = ms.scales[t - 2] if t >= 2 else side
    return dict(ms=ms, t=t, B=B, h=side, w=side, hp=prev, wp=prev, N=side * side,
                P=ms.prior_tokens(t), Lmax=ms.total_tokens, keep=args.keep)


def config_json(wd, n_gpus):
    ms = wd["ms"]
    return {
        "workload": f"{ms.name}: scale {wd['t']} ({wd['h']}x{wd['w']} = {wd['N']} tokens, {wd['P']} prior tokens), "
                    f"{ms.L} layers, width {ms.C}, {ms.heads} heads x {ms.dh}, MLP {ms.F}, V={synth.V_CODEBOOK}, "
                    f"batch {wd['B']} per GPU, keep ratio {wd['keep']}",
        "batch_per_gpu": wd["B"], "layers": ms.L, "tokens": wd["N"], "prior_tokens": wd["P"],
        "keep_ratio": wd["keep"], "l2": "inputs_larger_than_l2", "parallelism": f"replicas x{n_gpus}",
    }


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.path = tempfile.mktemp(suffix=".csv")
        self.proc = None
        try:
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(device_index), "-lms", "100"], stdout=self.fh,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.path)
        except OSError:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------ state
def build_state(wd, device, seed=0):
    """Random-init weights, prior K/V caches, previous residual caches and per-layer logits."""
    ms, B, N = wd["ms"], wd["B"], wd["N"]
    weights = [synth.block_weights(ms.C, ms.F, seed * 100 + j, device) for j in range(ms.L)]
    k_caches, v_caches = [], []
    for j in range(ms.L):
        k, v, _ = synth.kv_cache(B, wd["Lmax"], wd["P"], ms.C, seed * 1000 + 2 * j, device)
        k_caches.append(k)
        v_caches.append(v)
    kv_len0 = torch.full((ms.L, B), wd["P"], dtype=torch.int32, device=device)
    cache_prev = [synth.residual_cache(B, wd["hp"], wd["wp"], ms.C, seed * 10 + j, device) for j in range(ms.L)]
    a = synth.smooth_temperature_field(B, wd["h"], wd["w"], seed, a_lo=0.5, a_hi=6.0, device=device)
    beta = synth.layer_inverse_temperatures(ms.L, seed)
    logits = [synth.logits_from_temperature(a * float(beta[j]), synth.V_CODEBOOK, seed * 7 + j) for j in range(ms.L)]
    x_in = synth.activations(B, N, ms.C, seed + 5, device)
    return dict(weights=weights, k_caches=k_caches, v_caches=v_caches, kv_len0=kv_len0,
                kv_len=kv_len0.clone(), cache_prev=cache_prev, logits=logits, x_in=x_in)


def attention_flops(keeps, P, C):
    """4 * sum_b k_b * (P + k_b) * C for one layer (QK^T and PV, 2 flops per multiply-add)."""
    return sum(4.0 * int(k) * (P + int(k)) * C for k in keeps.tolist())


def peaks():
    try:
        p = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        return dict(hbm=float(p["hbm_gbs"]), tensor=float(p["bf16_tflops_sustained"]), source="measured")
    except Exception:
        return dict(hbm=6650.0, tensor=1400.0, source="fallback")


# ------------------------------------------------------------------- replicas (N > 1)
def max_over_ranks(ms: float, dist, device) -> float:
    """The job's time is the slowest rank's: all-reduce MAX of the per-rank device time. With
    dist None (one process) the value passes through."""
    if dist is None:
        return float(ms)
    tt = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def replica_throughput(world: int, units_per_rank: float, ms_per_step: float) -> float:
    """Whole-job throughput of `world` independent replicas (images are independent: no data-path
    collective; weak scaling): every rank processes units_per_rank per step, the step lasts as
    long as the slowest rank."""
    return world * units_per_rank / (ms_per_step / 1e3)


# ------------------------------------------------------------------------------ ours
def run_ours(args):
    import paper_2602_01345_b200 as nova
    from paper_2602_01345_b200 import pipeline

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    wd = workload_desc(args)
    ms, B, N = wd["ms"], wd["B"], wd["N"]

    ctx = nova.Context(local)
    st = build_state(wd, dev)
    fused = not args.two_call_layers
    runner = pipeline.PrunedScaleRunner(ctx, st["weights"], ms.heads, B, wd["h"], wd["w"], wd["Lmax"],
                                        st["k_caches"], st["v_caches"], st["kv_len"], st["cache_prev"],
                                        fused_restore=fused)
    sched = nova.SchedParams(force_act_scale=wd["t"], force_keep_ratio=wd["keep"])
    hbar_scale = torch.linspace(2.0, 7.0, wd["t"]).repeat(B, 1).contiguous()
    stream = torch.cuda.current_stream()

    def one_step():
        st["kv_len"].copy_(st["kv_len0"])          # every step starts from the same cache state
        return runner.run_scale(st["x_in"], st["logits"], sched, wd["t"], hbar_scale, stream=stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    torch.cuda.reset_peak_memory_stats()
    for _ in range(args.warmup):
        one_step()
    barrier()
    status = ctx.device_status()
    assert status == 0, f"device status after warm-up: {nova.STATUS_NAMES.get(status, status)}"

    clocks = ClockSampler(local)
    launches0 = pipeline.launch_count(ctx)
    # Event brackets inside the timed region go around the launches of the two contractions only (the
    # attention kernel and the GEMM kernel: one of them is the dominant kernel, which of the two is
    # known afterwards); every bracket costs two event records on the stream. The HBM-bound passes
    # get theirs in a few more steps after the timed region.
    pipeline.profile_begin(ctx, CONTRACTIONS)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        x_out, keeps = one_step()
    e1.record(stream)
    barrier()
    total_ms = e0.elapsed_time(e1)
    prof = pipeline.profile_end(ctx)
    launches = pipeline.launch_count(ctx) - launches0
    clk = clocks.stop()
    # the other kernels' brackets: same steps, after the timed region
    other_steps = min(3, args.steps)
    pipeline.profile_begin(ctx, [c for c in pipeline.profile_category_names(ctx) if c not in CONTRACTIONS])
    for _ in range(other_steps):
        one_step()
    barrier()
    prof_other = pipeline.profile_end(ctx)
    # per-step figures of both windows in one table: (summed ms, launches) scaled to args.steps steps
    for k, v in prof_other.items():
        if v[1]:
            prof[k] = (v[0] * args.steps / other_steps, v[1] * args.steps // other_steps)
    total_ms = max_over_ranks(total_ms, dist, dev)
    # device memory in use at its peak up to here: weights, K/V and residual caches, logits, activations
    # and the library's workspace (a torch tensor), i.e. everything the step needs resident
    peak_hbm_bytes = int(torch.cuda.max_memory_allocated())
    ms_per_step = total_ms / args.steps
    value = replica_throughput(world, B, ms_per_step)
    status = ctx.device_status()
    assert status == 0, f"device status after the timed region: {nova.STATUS_NAMES.get(status, status)}"
    assert bool(torch.isfinite(x_out.float()).all()), "the timed step produced non-finite outputs"

    # ---- rooflines from the events recorded around every launch inside the timed region. The two
    # contractions (the attention kernel and the GEMM kernel, four launches per layer) take about
    # equal shares of the step; `roofline` reports whichever took more time, `kernels` both.
    pk = peaks()
    default_shape = (args.workload == "c4_1024" and B == 4 and args.keep == 0.5 and wd["t"] == len(ms.scales))
    M = int(keeps[0].sum())
    kernels = {k: {"ms_per_step": round(v[0] / args.steps, 4), "launches_per_step": v[1] / args.steps,
                   "bracketed": "timed region" if k in CONTRACTIONS else f"{other_steps} more steps after the timed region"}
               for k, v in prof.items() if v[1]}
    attn_ms, attn_n = prof["attention"]
    attn_flops = attention_flops(keeps[0], wd["P"], ms.C)
    attn_tf = attn_flops / (attn_ms / attn_n * 1e-3) / 1e12 if attn_n else 0.0
    if attn_n:
        kernels["attention"]["tflops"] = round(attn_tf, 1)
    gemm_flops = {"gemm_qkv": 2.0 * M * 3 * ms.C * ms.C, "gemm_proj": 2.0 * M * ms.C * ms.C,
                  "gemm_fc1": 2.0 * M * ms.F * ms.C, "gemm_fc2": 2.0 * M * ms.F * ms.C}
    gemm_ms = gemm_n = 0.0
    for k, fl in gemm_flops.items():
        if k in kernels and prof[k][1]:
            kernels[k]["tflops"] = round(fl / (prof[k][0] / prof[k][1] * 1e-3) / 1e12, 1)
            gemm_ms += prof[k][0]
            gemm_n += prof[k][1]
    gemm_tf = sum(gemm_flops.values()) / (gemm_ms / (gemm_n / 4) * 1e-3) / 1e12 if gemm_n else 0.0

    traffic = ncu_traffic() if default_shape else {}

    def tensor_roofline(name, achieved, launches_per_layer, traffic_key):
        return {"kernel": name, "bound": "tensor", "achieved": round(achieved, 2), "peak": pk["tensor"],
                "unit": "TFLOP/s", "frac": round(achieved / pk["tensor"], 4),
                "frac_of_nominal": round(achieved / NOMINAL_PEAKS["tensor"], 4), "nominal_peak": NOMINAL_PEAKS["tensor"],
                "traffic": traffic.get(traffic_key),
                "launches_per_layer": launches_per_layer, "peak_source": pk["source"] + " (bf16 sustained)"}

    roof_attn = tensor_roofline("attention_kernel", attn_tf, 1, "attention")
    roof_gemm = tensor_roofline("gemm_bf16_tn_pair (qkv, proj, fc1, fc2)", gemm_tf, 4, "gemm")
    roofline = roof_attn if attn_ms >= gemm_ms else roof_gemm
    other_roofline = roof_gemm if attn_ms >= gemm_ms else roof_attn
    rows = B * N
    # HBM-bound passes: algorithmic bytes of all launches of a step over their summed event time.
    # entropy: per token V * 2 bytes read + 4 written; select: per token a 4-byte key read and a 4-byte
    # index written; restore: kept row = y and x_in read, x_out and cache_out written (4 rows; when the
    # block's last GEMM writes the kept rows itself, restore touches the pruned rows only), pruned row =
    # x_in read, x_out and cache_out written (3 rows), plus the low-resolution cache once.
    ent_bytes_step = ms.L * rows * (synth.V_CODEBOOK * 2 + 4)
    sel_bytes_step = ms.L * rows * 8
    kept_rows_in_restore = 0 if fused else M
    restore_bytes = (kept_rows_in_restore * 4 + (rows - M) * 3) * ms.C * 2 + B * wd["hp"] * wd["wp"] * ms.C * 2
    for key, step_bytes in (("entropy_rows", ent_bytes_step), ("select_topk", sel_bytes_step),
                            ("restore", restore_bytes * ms.L)):
        if prof.get(key, (0, 0))[1]:
            kernels[key]["gbs"] = round(step_bytes * args.steps / (prof[key][0] * 1e-3) / 1e9, 1)
            kernels[key]["bytes_per_launch"] = int(step_bytes * args.steps / prof[key][1])
    # The entropy pass once more outside the timed region, back to back between one pair of events,
    # with and without the per-image means.
    ent_buf = torch.empty((ms.L, B, N), dtype=torch.float32, device=dev)
    mean_buf = torch.empty((ms.L, B), dtype=torch.float32, device=dev)
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for with_mean in (True, False):
        torch.cuda.synchronize()
        b0.record(stream)
        for _ in range(3):
            nova.nova_scale_entropy_layers(ctx, st["logits"], ent_buf, mean_buf if with_mean else None, stream=stream)
        b1.record(stream)
        torch.cuda.synchronize()
        us = b0.elapsed_time(b1) * 1e3 / 3
        key = "gbs_back_to_back" if with_mean else "gbs_back_to_back_no_mean"
        kernels["entropy_rows"][key] = round(ent_bytes_step / us / 1e3, 1)
    # Both forms of a layer (one nova_pruned_layer_forward call, or block + restore as two calls) on the
    # same inputs, timed alike: no per-kernel event brackets here, which cost the timed region above two
    # event records per launch.
    other = pipeline.PrunedScaleRunner(ctx, st["weights"], ms.heads, B, wd["h"], wd["w"], wd["Lmax"], st["k_caches"],
                                       st["v_caches"], st["kv_len"], st["cache_prev"], fused_restore=not fused)
    form_ms, form_out = {}, {}
    for name, rn in (("timed", runner), ("other", other)):
        for it in range(2 + args.steps):
            if it == 2:
                torch.cuda.synchronize()
                b0.record(stream)
            st["kv_len"].copy_(st["kv_len0"])
            form_out[name], _ = rn.run_scale(st["x_in"], st["logits"], sched, wd["t"], hbar_scale, stream=stream)
        b1.record(stream)
        torch.cuda.synchronize()
        form_ms[name] = b0.elapsed_time(b1) / args.steps
    layer_forms = {"timed": "one call per layer (nova_pruned_layer_forward)" if fused else
                            "two calls per layer (nova_pruned_block_forward + nova_restore_from_cache)",
                   "ms_per_step_one_call": round(form_ms["timed" if fused else "other"], 4),
                   "ms_per_step_two_calls": round(form_ms["other" if fused else "timed"], 4),
                   "note": "both without the per-kernel event brackets of the timed region",
                   "same_result": bool(torch.equal(form_out["timed"], form_out["other"]))}
    del other
    head_entropy = device_schedule = None
    if not args.no_next:
        # Entropy fused with the codebook head (the step before the path: hidden states -> entropy, the
        # 8 KiB/token of logits never stored), timed back to back over 8 calls outside the timed region.
        head_w = synth.randn_bf16((synth.V_CODEBOOK, ms.C), 991, dev, std=3.0 / ms.C ** 0.5)
        hidden = [synth.activations(B, N, ms.C, 900 + i, dev) for i in range(4)]
        for _ in range(2):
            nova.nova_head_entropy(ctx, hidden[0], head_w, None, ent_buf[0], mean_buf[0], stream=stream)
        torch.cuda.synchronize()
        b0.record(stream)
        for i in range(8):
            nova.nova_head_entropy(ctx, hidden[i % 4], head_w, None, ent_buf[0], mean_buf[0], stream=stream)
        b1.record(stream)
        torch.cuda.synchronize()
        head_us = b0.elapsed_time(b1) * 1e3 / 8
        head_tf = 2.0 * rows * ms.C * synth.V_CODEBOOK / head_us / 1e6
        head_entropy = {"us_per_call": round(head_us, 1), "tflops": round(head_tf, 1),
                        "frac_of_tensor_peak": round(head_tf / pk["tensor"], 4),
                        "logits_bytes_not_written_or_read": int(2 * rows * synth.V_CODEBOOK * 2)}
        assert ctx.device_status() == 0, "device status after the head-entropy timing"
        # The same step with every decision left on the device (Eq. 8-13 in a kernel, kept counts read
        # from device memory, launches sized by the upper bound B*N): issued eagerly, and recorded once
        # in a CUDA graph and replayed. Same inputs and buffers as the timed region above.
        hist_dev = hbar_scale.t().contiguous().to(dev)
        drun = pipeline.DeviceScaleRunner(ctx, st["weights"], ms.heads, B, wd["h"], wd["w"], wd["Lmax"], st["k_caches"],
                                          st["v_caches"], st["kv_len"], st["cache_prev"], sched, wd["t"], hist_dev,
                                          synth.V_CODEBOOK, x_in=st["x_in"], layer_logits=st["logits"], scale_entropy=False,
                                          fused_restore=fused)
        st["kv_len"].copy_(st["kv_len0"])
        l0 = pipeline.launch_count(ctx)
        drun.capture()
        dev_launches = (pipeline.launch_count(ctx) - l0) // 2          # one eager pass + one recorded pass
        dev_ms = {}
        for mode in ("eager", "graph"):
            for it in range(args.warmup + args.steps):
                if it == args.warmup:
                    torch.cuda.synchronize()
                    b0.record(stream)
                st["kv_len"].copy_(st["kv_len0"])
                if mode == "eager":
                    drun.enqueue(stream=stream)
                else:
                    drun.replay()
            b1.record(stream)
            torch.cuda.synchronize()
            dev_ms[mode] = b0.elapsed_time(b1) / args.steps
        assert ctx.device_status() == 0, "device status after the device-driven timing"
        same = bool(torch.equal(drun.x_out, x_out)) and bool(torch.equal(drun.keep.cpu(), torch.stack(keeps)))
        max_diff = float((drun.x_out.float() - x_out.float()).abs().max())
        device_schedule = {"ms_per_step_eager": round(dev_ms["eager"], 4), "ms_per_step_graph": round(dev_ms["graph"], 4),
                           "ms_per_step_host_driven": round(ms_per_step, 4), "launches_per_step": int(dev_launches),
                           "host_syncs_per_step": 0, "equals_host_driven_result": same,
                           "max_abs_diff_vs_host_driven": max_diff}
    for k in kernels:
        if "gbs" in kernels[k]:
            kernels[k]["frac_of_hbm_peak"] = round(kernels[k]["gbs"] / pk["hbm"], 4)
            kernels[k]["frac_of_nominal_hbm"] = round(kernels[k]["gbs"] / NOMINAL_PEAKS["hbm"], 4)
        if "tflops" in kernels[k]:
            kernels[k]["frac_of_tensor_peak"] = round(kernels[k]["tflops"] / pk["tensor"], 4)
            kernels[k]["frac_of_nominal_tensor"] = round(kernels[k]["tflops"] / NOMINAL_PEAKS["tensor"], 4)
    kernels["entropy_rows"]["frac_of_hbm_peak_back_to_back"] = round(kernels["entropy_rows"]["gbs_back_to_back"] / pk["hbm"], 4)

    out = {
        "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_json(wd, world), "clocks": clk, "gpu_launches": int(launches),
        "tokens_per_s": round(world * B * N / (ms_per_step / 1e3), 1), "peak_hbm_bytes": peak_hbm_bytes,
        "roofline": roofline, "roofline_second": other_roofline, "kernels": kernels,
        "layer_call_forms": layer_forms,
        "next_head_entropy": head_entropy, "next_device_schedule": device_schedule,
    }

    # ---- end to end: inputs start in pinned host memory, result read back every step
    if not args.no_e2e:
        out["e2e"] = run_e2e(args, wd, st, runner, sched, hbar_scale, barrier, dist, dev, world)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wd, st, keeps)
    if dist is not None:
        dist.destroy_process_group()
    return out if rank == 0 else None


ALL_CONFIGS = (
    [("c1_single_step", None, 0.5), ("c2_var_d16_256", None, 0.5), ("c3_var_d30_512", None, 0.5)] +
    [("c4_1024", b, k) for b in (1, 4) for k in (0.25, 0.5, 0.75)] + [("c5_2048", None, 0.2)])


def run_all_configs(args):
    """The stated configurations one after the other in this process, device-resident timing only."""
    import copy
    import gc
    for wl, batch, keep in ALL_CONFIGS:
        a = copy.copy(args)
        a.workload, a.batch, a.keep = wl, batch, keep
        a.no_e2e = a.no_cpu_baseline = True
        out = run_ours(a)
        if out is not None:
            print(json.dumps(out), flush=True)
        del out
        gc.collect()
        torch.cuda.empty_cache()


def run_e2e(args, wd, st, runner, sched, hbar_scale, barrier, dist, dev, world):
    ms, B, N = wd["ms"], wd["B"], wd["N"]
    L = ms.L
    host_x = st["x_in"].cpu().pin_memory()
    host_logits = [t.cpu().pin_memory() for t in st["logits"]]
    host_out = torch.empty_like(host_x).pin_memory()
    dev_x = torch.empty_like(st["x_in"])
    dev_logits = [torch.empty_like(t) for t in st["logits"]]
    copy_stream = torch.cuda.Stream()
    main = torch.cuda.current_stream()
    h2d = host_x.numel() * 2 + sum(t.numel() * 2 for t in host_logits)
    d2h = host_out.numel() * 2

    def e2e_step():
        st["kv_len"].copy_(st["kv_len0"])
        copy_stream.wait_stream(main)               # the previous step no longer reads the device buffers
        ready = []
        with torch.cuda.stream(copy_stream):
            dev_x.copy_(host_x, non_blocking=True)
            x_ready = torch.cuda.Event()
            x_ready.record(copy_stream)
            for j in range(L):
                dev_logits[j].copy_(host_logits[j], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(copy_stream)
                ready.append(ev)
        main.wait_event(x_ready)
        x_out, _ = runner.run_scale(dev_x, dev_logits, sched, wd["t"], hbar_scale, stream=main, logits_ready=ready)
        host_out.copy_(x_out, non_blocking=True)
        main.synchronize()

    for _ in range(2):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(main)
    for _ in range(args.steps):
        e2e_step()
    e1.record(main)
    barrier()
    wall_ms = (time.perf_counter() - t0) * 1e3
    dev_ms = e0.elapsed_time(e1)
    t_ms = max(wall_ms, dev_ms)
    t_ms = max_over_ranks(t_ms, dist, dev)
    per = t_ms / args.steps
    return {"value": round(world * B / (per / 1e3), 3), "unit": UNIT, "ms_per_step": round(per, 3),
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "note": "pinned host x_in and per-layer logits uploaded on a copy stream overlapped with compute; x_out read back"}


# ---------------------------------------------------------------------- CPU baseline (oracle)
def oracle_sample_sizes(threads: int):
    """Row counts of one oracle sample: enough rows for every OpenMP thread to stay busy (the oracle
    parallelises over rows only)."""
    return dict(rows_entropy=max(256, 32 * threads), rows_block=4 * threads)


def oracle_sample(wd, st, keeps):
    """Times the oracle, as it stands, on one layer of one image and extrapolates to the whole
    pruned scale: entropy on a row sample, selection on the full map, K/V of every kept token
    (exact), attention + MLP on a row sample (4 rows per thread, timed as the difference between a
    call with those rows and a call with none), restore on the full map. Returns (seconds per
    image-layer, parts, threads, sizes)."""
    import numpy as np

    import oracle
    ms, N = wd["ms"], wd["N"]
    f32 = synth.to_f32_numpy
    threads = oracle.num_threads()
    sz = oracle_sample_sizes(threads)
    rows_entropy = min(sz["rows_entropy"], N)
    t = {}
    logits = f32(st["logits"][0][0:1, :rows_entropy])
    t0 = time.perf_counter()
    oracle.scale_entropy(logits)
    t["entropy"] = (time.perf_counter() - t0) * (N / rows_entropy)
    ent_full = np.random.default_rng(0).random((1, N)).astype(np.float32)
    k = int(keeps[0][0])
    rows_block = min(sz["rows_block"], k)
    t0 = time.perf_counter()
    keep_idx, prune_idx, cu, _ = oracle.select_topk(ent_full, [k])
    t["select"] = time.perf_counter() - t0
    wts = {n: f32(v) for n, v in st["weights"][0].items()}
    x = f32(st["x_in"][0:1])
    kc, vc = f32(st["k_caches"][0][0:1]), f32(st["v_caches"][0][0:1])
    kv_len = np.array([wd["P"]], np.int32)
    none = np.zeros(0, np.int32)
    # first call untimed: it also pays for the first touch of the converted K/V caches
    oracle.pruned_block_forward(wts, 1e-6, ms.heads, x, keep_idx, cu, kc, vc, kv_len, rows=none)
    t0 = time.perf_counter()
    oracle.pruned_block_forward(wts, 1e-6, ms.heads, x, keep_idx, cu, kc, vc, kv_len, rows=none)
    t["block_kv"] = time.perf_counter() - t0
    rows = np.linspace(0, k - 1, rows_block).astype(np.int32)
    t0 = time.perf_counter()
    oracle.pruned_block_forward(wts, 1e-6, ms.heads, x, keep_idx, cu, kc, vc, kv_len, rows=rows)
    t["block_rows"] = max(time.perf_counter() - t0 - t["block_kv"], 0.0) * (k / rows_block)
    y_full = np.zeros((k, ms.C), np.float32)
    t0 = time.perf_counter()
    oracle.restore_from_cache(x, y_full, keep_idx, prune_idx, cu, f32(st["cache_prev"][0][0:1]), wd["h"], wd["w"])
    t["restore"] = time.perf_counter() - t0
    return sum(t.values()), t, threads, dict(rows_entropy=rows_entropy, rows_block=rows_block, kept=k)


def sample_text(sizes, threads, L):
    return (f"one layer of one image: entropy on {sizes['rows_entropy']} rows, top-k on the full map, K/V of all "
            f"{sizes['kept']} kept tokens, attention+MLP on {sizes['rows_block']} kept rows "
            f"({sizes['rows_block'] // max(threads, 1)} per thread, all {threads} threads busy), restore on the full map; "
            f"each part scaled to the full row count, then x{L} layers")


def cpu_baseline(wd, st, keeps, repeats=3):
    """The oracle on the host cores: `repeats` samples, the median per part."""
    runs = [oracle_sample(wd, st, keeps) for _ in range(repeats)]
    parts = {k: statistics.median(r[1][k] for r in runs) for k in runs[0][1]}
    totals = sorted(r[0] for r in runs)
    threads, sizes = runs[0][2], runs[0][3]
    ms = wd["ms"]
    sec_per_image = sum(parts.values()) * ms.L
    return {"value": round(1.0 / sec_per_image, 6), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": sample_text(sizes, threads, ms.L) + f"; median of {repeats} samples",
            "seconds_per_image_layer": {k: round(v, 3) for k, v in parts.items()},
            "spread_seconds_per_image_layer": [round(totals[0], 3), round(totals[-1], 3)]}


def run_reference(args):
    """The oracle as the reference arm: same metric and workload, bounded sample per step (the same
    sample, of the same size, as the `cpu_baseline` leg of the other arm)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wd = workload_desc(args)
    ms = wd["ms"]
    wd_small = dict(wd, B=1)
    st = build_state_cpu_one_layer(wd_small)
    k = wd["N"] - int((1.0 - wd["keep"]) * wd["N"])
    keeps = [torch.tensor([k], dtype=torch.int32)]
    times = []
    threads, sizes = 1, {}
    for i in range(args.warmup + args.steps):
        per_image_layer, _, threads, sizes = oracle_sample(wd_small, st, keeps)
        if i >= args.warmup:
            times.append(per_image_layer * ms.L)
    sec_per_image = statistics.median(times)
    value = 1.0 / sec_per_image
    sample = "per step: " + sample_text(sizes, threads, ms.L) + f"; median of {len(times)} steps"
    out = {"impl": "reference", "metric": METRIC, "value": round(value, 6), "unit": UNIT,
           "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": round(sec_per_image * wd["B"] * 1e3, 1), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config_json(wd, 1),
           "cpu_baseline": {"value": round(value, 6), "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                            "spread_seconds_per_image": [round(min(times), 1), round(max(times), 1)]},
           "e2e": {"value": round(value, 6), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def build_state_cpu_one_layer(wd):
    """Layer-0 inputs of the workload for one image, generated on the CPU."""
    ms, N = wd["ms"], wd["N"]
    a = synth.smooth_temperature_field(1, wd["h"], wd["w"], 0)
    k, v, _ = synth.kv_cache(1, wd["Lmax"], wd["P"], ms.C, 0, "cpu")
    return dict(weights=[synth.block_weights(ms.C, ms.F, 0, "cpu")], k_caches=[k], v_caches=[v],
                cache_prev=[synth.residual_cache(1, wd["hp"], wd["wp"], ms.C, 0, "cpu")],
                logits=[synth.logits_from_temperature(a[:, :4096].contiguous(), synth.V_CODEBOOK, 0)],
                x_in=synth.activations(1, N, ms.C, 5, "cpu"))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    elif a.all_configs:
        run_all_configs(a)
    else:
        res = run_ours(a)
        if res is not None:
            print(json.dumps(res))

#!/usr/bin/env python
"""Benchmark of the hot path: frames/s through (plan refresh every k-th layer) + merge +
global attention + unmerge on a synthetic VGGT-shaped sequence.

A step is one global layer: when ``step % recompute_interval == 0`` the merge plan is
rebuilt first (the Grad map once, at step 0), then merge -> global attention over the
merged tokens -> unmerge with the residual, and the result feeds the next layer.  With the
default K = 6 the timed region holds exactly one refresh period, i.e. every step of the
path runs inside it.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C5] [--impl ours|reference]

N > 1 (torchrun): the path does not shard, so every rank runs an independent replica of
the workload (its own seeded sequence); no data-path collective exists.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from synthdata import WORKLOADS, make_attention_weights, make_block_weights, make_images, make_tokens

import hashlib

METRIC = "frames/s through merge+global-attn+unmerge (plan refreshed every 6th layer)"
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the attention core per layer on
# workload C5, summed over the layer's key-chunk launches, from one single-pass ncu capture
# (profiles/flash_attention_C5_dram.md).  Reported only while the kernel source is the one that was
# measured.
ATTENTION_TRAFFIC_C5 = {"bytes_per_layer": 34.65e9 + 17.60e9, "kernel_sha256": "dce9e561e33d972a66c4798f3eb9686614976653cbcabe9afecc16fd9265da67"}


def _attention_source_hash() -> str:
    h = hashlib.sha256()
    for name in ("attention.cu", "common.cuh"):
        with open(os.path.join(ROOT, "paper_2512_04939_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()
UNIT = "frames/s"


def _measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return dict(hbm_gbs=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------
# CPU oracle leg (the reported baseline, and the --impl reference arm)
# ----------------------------------------------------------------------------------------------
# The oracle cannot run a 1000-frame layer (the attention core alone is 1.1e15 flops), so it is timed
# on bounded samples OF THE TRUE-SIZE PROBLEM and extrapolated by rows/s x rows:
#   * the two quadratic steps on seeded row samples against the whole sequence: `match_rows` src rows
#     x all anchors, `attn_rows` query rows x all M keys for `attn_heads` heads (one head at a time);
#   * the projections on `proj_rows` rows with the full weight matrices;
#   * the steps that cost the same per frame whatever the length (Grad map, Var map, GA map +
#     partition, merge, unmerge) on a sub-sequence of `linear_frames` frames, x F / linear_frames
#     (a float64 copy of the whole token matrix is 8.5 GB at 1000 frames);
#   * selection + index build at full size (on seeded similarities: its cost does not depend on them).
CPU_SAMPLE = dict(match_rows=2048, attn_rows=256, attn_heads=4, proj_rows=8192, linear_frames=64)
REF_SAMPLE = dict(match_rows=256, attn_rows=64, attn_heads=1, proj_rows=1024, linear_frames=16)


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def prepare_oracle_sample(wl, images, tokens, weights, sample):
    """Everything the timed oracle calls need, drawn once (nothing here is timed): the sub-sequence
    for the per-frame steps, a full-size class array from the oracle's own partition of a seeded
    random score map (true counts, anchors of every frame), the sampled src rows with all anchors as
    one compact float64 matrix, and K / V of the sampled heads for all M rows (the first M token
    rows stand in for the merged rows: same shape and distribution, and timing does not depend on
    the values)."""
    import oracle as O

    rng = np.random.default_rng(wl.seed + 31)
    t_tok, d = wl.tokens_per_frame, 1024
    lf = min(sample["linear_frames"], wl.frames)
    sz = O.derived_sizes(wl.frames, wl.grid_h, wl.grid_w, merge_ratio=wl.merge_ratio)
    data = dict(sizes=sz, linear_frames=lf)
    data["images_sub"] = images[:lf].cpu().numpy()
    data["x_sub"] = _f64(tokens[:lf * t_tok])
    cls = O.partition(rng.random((wl.frames, wl.grid_h, wl.grid_w)))
    src_idx, dst_idx = np.flatnonzero(cls == O.CLS_SRC), np.flatnonzero(cls == O.CLS_DST)
    data["cls"] = cls
    n_rows = min(sample["match_rows"], src_idx.size)
    rows = np.sort(rng.choice(src_idx.size, n_rows, replace=False))
    dev = tokens.device
    sel = torch.from_numpy(np.concatenate([dst_idx, src_idx[rows]])).to(dev)
    data["x_match"] = _f64(tokens[sel])
    data["match_src"] = dst_idx.size + np.arange(n_rows)
    data["match_dst"] = np.arange(dst_idx.size)
    data["best_dst_full"] = dst_idx[rng.integers(0, dst_idx.size, src_idx.size)]
    data["best_sim_full"] = rng.random(src_idx.size)
    # K and V of the sampled heads for all M rows, Q for the sampled rows (same projection)
    m = sz["M"]
    heads = list(range(0, 16, max(1, 16 // sample["attn_heads"])))[:sample["attn_heads"]]
    w_qkv, b_qkv = _f64(weights[0]), _f64(weights[1])
    per_head = []
    for h in heads:
        cols = np.concatenate([np.arange(64) + 64 * h, d + np.arange(64) + 64 * h, 2 * d + np.arange(64) + 64 * h])
        parts = []
        for r0 in range(0, m, 65536):
            parts.append(O.linear(_f64(tokens[r0:min(m, r0 + 65536)]), w_qkv[cols], b_qkv[cols]))
        per_head.append(np.concatenate(parts))
    data["qkv_heads"] = per_head
    data["attn_rows"] = np.sort(rng.choice(m, min(sample["attn_rows"], m), replace=False))
    data["x_proj"] = _f64(tokens[:min(sample["proj_rows"], m)])
    data["weights"] = [_f64(u) for u in weights]
    return data


def oracle_sampled_layer(wl, data):
    """One pass of the timed oracle calls.  Returns seconds per step, already scaled to the full
    sequence, and the top-1 / top-2 margins of the sampled matches."""
    import oracle as O

    sz, lf = data["sizes"], data["linear_frames"]
    per_frame = wl.frames / lf
    tic = time.perf_counter
    t = {}
    t0 = tic(); grad = O.grad_map(data["images_sub"]); t["grad_map"] = (tic() - t0) * per_frame
    t0 = tic(); var = O.var_map(data["x_sub"], lf, wl.grid_h, wl.grid_w); t["var_map"] = (tic() - t0) * per_frame
    t0 = tic(); cls_sub = O.partition(O.ga_map(grad, var)); t["partition"] = (tic() - t0) * per_frame
    t0 = tic()
    _, sim1, sim2 = O.match(data["x_match"], data["match_src"], data["match_dst"])
    t["match"] = (tic() - t0) * sz["n_src"] / data["match_src"].size
    t0 = tic()
    O.select_and_index(data["cls"], data["best_dst_full"], data["best_sim_full"], sz["R"])
    t["index_build"] = tic() - t0
    # merge / unmerge on the sub-sequence, with a plan of its own (every src token of the sub-sequence
    # merged into a seeded anchor of the sub-sequence)
    src_s, dst_s = np.flatnonzero(cls_sub == O.CLS_SRC), np.flatnonzero(cls_sub == O.CLS_DST)
    rng = np.random.default_rng(7)
    dst_of, size, _ = O.select_and_index(cls_sub, dst_s[rng.integers(0, dst_s.size, src_s.size)], rng.random(src_s.size),
                                         src_s.size)
    t0 = tic(); xm = O.merge(data["x_sub"], dst_of, size.size); t["merge"] = (tic() - t0) * per_frame
    t0 = tic(); O.unmerge(xm, dst_of, data["x_sub"]); t["unmerge"] = (tic() - t0) * per_frame
    w = data["weights"]
    rows_scale = sz["M"] / data["x_proj"].shape[0]
    t0 = tic(); O.linear(data["x_proj"], w[0], w[1]); t["qkv_proj"] = (tic() - t0) * rows_scale
    t0 = tic(); O.linear(data["x_proj"], w[2], w[3]); t["out_proj"] = (tic() - t0) * rows_scale
    t0 = tic()
    for qkv_h in data["qkv_heads"]:
        O.attention_core(qkv_h, heads=1, rows=data["attn_rows"])
    t["attention"] = (tic() - t0) * (sz["M"] / data["attn_rows"].size) * (16 / len(data["qkv_heads"]))
    return t, sim1 - sim2


def frames_per_s_from_steps(t, frames, interval):
    """frames / (layer + plan / interval): the plan steps are amortised over the refresh interval (the
    Grad map, computed once per sequence, is left out as in the GPU figure's steady state)."""
    plan = t["var_map"] + t["partition"] + t["match"] + t["index_build"]
    layer = t["merge"] + t["qkv_proj"] + t["attention"] + t["out_proj"] + t["unmerge"]
    return frames / (layer + plan / interval)


def sample_description(wl, sample, data):
    sz = data["sizes"]
    return (f"oracle (float64 numpy) on bounded samples of the true-size {wl.name} problem, extrapolated as rows/s x rows: "
            f"matching {data['match_src'].size} of {sz['n_src']} src rows x all {sz['n_dst']} anchors; attention core "
            f"{data['attn_rows'].size} of {sz['M']} query rows x all {sz['M']} keys, {len(data['qkv_heads'])} of 16 heads; "
            f"projections {data['x_proj'].shape[0]} of {sz['M']} rows; Grad map, Var map, partition, merge, unmerge on "
            f"{data['linear_frames']} of {wl.frames} frames (x F/{data['linear_frames']}); selection + index build at full "
            f"size; plan amortised over {wl.recompute_interval} layers")


def margin_histogram(margin):
    return {"rows": int(margin.size), "below_1e-5": float((margin < 1e-5).mean()), "below_1e-4": float((margin < 1e-4).mean()),
            "below_1e-3": float((margin < 1e-3).mean()), "median": float(np.median(margin))}


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        n = os.cpu_count() or 1
    return int(n)


def run_cpu_baseline(wl, images, tokens, weights):
    data = prepare_oracle_sample(wl, images, tokens, weights, CPU_SAMPLE)
    t0 = time.perf_counter()
    t, margin = oracle_sampled_layer(wl, data)
    spent = time.perf_counter() - t0
    return {
        "value": frames_per_s_from_steps(t, wl.frames, wl.recompute_interval), "unit": UNIT, "cores": cpu_threads(),
        "kind": "oracle", "sample": sample_description(wl, CPU_SAMPLE, data) + f" ({spent:.1f} s of CPU time)",
        "extrapolated": True, "seconds_per_step_full_size": {k: round(v, 2) for k, v in t.items()},
        "match_margin_top1_top2": dict(margin_histogram(margin),
                                       note="sampled src rows; anchors from the oracle's partition of a seeded random score map"),
    }


def run_reference(args, wl):
    """--impl reference: the CPU oracle as it stands, each step a bounded sample of the true-size workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    dev = "cuda" if torch.cuda.is_available() else "cpu"  # the seeded input generator only; the oracle runs on the host
    images = make_images(wl, dev)
    tokens = make_tokens(wl, images)
    weights = make_attention_weights(wl, 0)
    data = prepare_oracle_sample(wl, images, tokens, weights, REF_SAMPLE)
    del images, tokens
    for _ in range(args.warmup):
        oracle_sampled_layer(wl, data)
    times = []
    t_all = time.perf_counter()
    for _ in range(args.steps):
        times.append(oracle_sampled_layer(wl, data)[0])
    wall = time.perf_counter() - t_all
    mean = {k: float(np.mean([t[k] for t in times])) for k in times[0]}
    value = frames_per_s_from_steps(mean, wl.frames, wl.recompute_interval)
    sample = "each step: " + sample_description(wl, REF_SAMPLE, data)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * wall / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(wl, data["sizes"]["N"], data["sizes"]["M"]), "sample": sample,
                   "extrapolated": True},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_name(wl, n, m):
    """One string for `config.workload`, the same in both arms."""
    return (f"{wl.name}: {wl.frames} frames {wl.img_w}x{wl.img_h}, N={n} tokens, M={m} merged, D=1024, "
            f"16 heads x 64, merge ratio {wl.merge_ratio}, plan refresh every {wl.recompute_interval} layers")


# ----------------------------------------------------------------------------------------------
# rank plumbing (replicas only: no data-path collective, just the timing reduction)
# ----------------------------------------------------------------------------------------------
def max_over_ranks(ms: float, world: int, device) -> float:
    """Slowest rank's time: the job is done when the last replica is."""
    if world <= 1:
        return float(ms)
    import torch.distributed as dist

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_frames_per_s(frames: int, steps: int, world: int, ms: float) -> float:
    """Whole-job throughput: every rank pushes its own `frames`-frame sequence through `steps` layers."""
    return world * frames * steps / (ms / 1e3)


def rank_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own sequence."""
    return base_seed + 17 * rank


# ----------------------------------------------------------------------------------------------
# the CUDA path
# ----------------------------------------------------------------------------------------------
def run_ours(args, wl):
    import torch.distributed as dist

    import paper_2512_04939_b200 as pkg

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    wl_rank = dataclasses.replace(wl, seed=rank_seed(wl.seed, rank))
    peaks = _measured_peaks()

    images = make_images(wl_rank, dev)
    tokens = make_tokens(wl_rank, images)
    ctx = pkg.LiteVGGT(wl.frames, wl.grid_h, wl.grid_w, wl.merge_ratio, device=local,
                       recompute_interval=wl.recompute_interval)
    n, m, d = ctx.n_tokens, ctx.n_merged, ctx.dim
    n_layers = max(args.steps, args.warmup, 1)
    weights = [[t.to(dev) for t in make_attention_weights(wl, layer)] for layer in range(n_layers)]
    xm = torch.empty(m, d, dtype=torch.bfloat16, device=dev)
    ym = torch.empty(m, d, dtype=torch.bfloat16, device=dev)
    bufs = [torch.empty(n, d, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    state = {"plan": None, "grad": None}

    def run_steps(count):
        cur = tokens
        for idx in range(count):
            if idx % wl.recompute_interval == 0:
                if idx == 0:
                    state["grad"] = ctx.grad_map(images)
                state["plan"] = ctx.merge_plan(cur, state["grad"], state["plan"])
            ctx.merge(state["plan"], cur, xm)
            ctx.global_attn(xm, *weights[idx], out=ym)
            nxt = bufs[idx & 1]
            ctx.unmerge(state["plan"], ym, cur, out=nxt)
            cur = nxt
        return cur

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    run_steps(args.warmup)
    ctx.poll()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ctx.timers_reset()
    launches0 = ctx.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    run_steps(args.steps)
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ctx.poll()
    timers = ctx.timers_read()
    ms = max_over_ranks(ms, world, dev)
    value = aggregate_frames_per_s(wl.frames, args.steps, world, ms)

    # ---- end to end through the host-buffer entry point (same schedule, same weights)
    # Every step is an independent batch: it uploads its own input from pinned memory and downloads its
    # own result; the entry point runs the copies on the context's copy streams, so they overlap the
    # neighbouring steps' kernels.  All of it - every copy included - lies inside the timed region.
    x_host = [torch.empty(n, d, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    out_host = [torch.empty(n, d, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    for buf in x_host:
        buf.copy_(tokens)
    e2e_plan = {"plan": None}

    def run_host_steps(count):
        for idx in range(count):
            grad = state["grad"] if idx % wl.recompute_interval == 0 else None
            e2e_plan["plan"] = ctx.global_layer_host_pipelined(e2e_plan["plan"], x_host[idx & 1], *weights[idx],
                                                               out_host[idx & 1], grad=grad)
        ctx.host_drain()
        torch.cuda.current_stream().synchronize()

    run_host_steps(2)
    barrier()
    t0 = time.perf_counter()
    ev0.record()
    run_host_steps(args.steps)
    ev1.record()
    barrier()
    e2e_ms = max(ev0.elapsed_time(ev1), 1e3 * (time.perf_counter() - t0))  # device span or host wall clock
    e2e_ms = max_over_ranks(e2e_ms, world, dev)
    ctx.poll()
    e2e_value = aggregate_frames_per_s(wl.frames, args.steps, world, e2e_ms)

    # ---- per-step statistics: every step of the path at least ten times (the attention layer, a
    # second per call at 1000 frames, five), device time of each call from the library's stopwatches;
    # the clocks are sampled alongside so that a time can be read as time x clock
    ctx.timers_reset()
    stats_sampler = ClockSampler(local)
    if rank == 0:
        stats_sampler.start()
    for _ in range(10):
        ctx.grad_map(images)
        ctx.merge_plan(tokens, state["grad"], state["plan"])
        ctx.merge(state["plan"], tokens, xm)
        ctx.unmerge(state["plan"], ym, tokens, out=bufs[0])
    attn_reps = 10 if m <= 100_000 else 5
    for i in range(attn_reps):
        ctx.global_attn(xm, *weights[i % len(weights)], out=ym)
    ctx.poll()
    step_samples = ctx.timers_samples()
    stats_clocks = stats_sampler.stop() if rank == 0 else None
    stats_mhz = stats_clocks["sm_mhz"] if stats_clocks else None

    # ---- the E4M3 variant of the attention operands, beside bf16 (same rows, same weights)
    fp8 = None
    if not args.no_fp8:
        ctx8 = pkg.LiteVGGT(wl.frames, wl.grid_h, wl.grid_w, wl.merge_ratio, device=local, qkv_dtype=1)
        ctx8.global_attn(xm, *weights[0], out=ym)
        ctx8.poll()
        ctx8.timers_reset()
        for i in range(attn_reps):
            ctx8.global_attn(xm, *weights[i % len(weights)], out=ym)
        ctx8.poll()
        s8 = ctx8.timers_samples()
        ctx8.close()
        core, quant = float(np.median(s8["attention"])), float(np.median(s8["qkv_quantize"]))
        fp8 = {"attention_core_ms_median": round(core, 3), "attention_core_ms_best": round(min(s8["attention"]), 3),
               "quantize_ms_median": round(quant, 3), "samples": len(s8["attention"]),
               "TFLOP/s": round(4.0 * m * m * d / (core * 1e-3) / 1e12, 1),
               "note": "qkv_dtype = 1: Q, K, V and the probabilities in E4M3, both products kind::f8f6f4; flops counted "
                       "as for bf16 (4 M^2 D); parity: tests/test_gpu_parity.py::test_fp8_attention_variant"}

    block = None
    if args.block:
        # One aggregator block (Sec. 3.1), pre-norm: x += frame_attn(LN x); x += MLP(LN x);
        # x += unmerge(global_attn(merge(LN x))); x += MLP(LN x).  Plan refreshed every k-th block.
        bw = make_block_weights(wl, 0, dev)
        bw2 = make_block_weights(wl, 1, dev)
        xn = torch.empty(n, d, dtype=torch.bfloat16, device=dev)
        cur, nxt = bufs[0], bufs[1]
        cur.copy_(tokens)
        bstate = {"plan": state["plan"]}

        def run_blocks(count):
            a, b_ = cur, nxt
            for idx in range(count):
                ctx.layernorm(a, *bw["ln1"], out=xn)
                ctx.frame_attn(xn, *bw["attn"], residual=a, out=b_)
                ctx.layernorm(b_, *bw["ln2"], out=xn)
                ctx.mlp(xn, *bw["mlp"], residual=b_, out=a)
                ctx.layernorm(a, *bw2["ln1"], out=xn)
                if idx % wl.recompute_interval == 0:
                    bstate["plan"] = ctx.merge_plan(xn, state["grad"], bstate["plan"])
                ctx.merge(bstate["plan"], xn, xm)
                ctx.global_attn(xm, *weights[idx % len(weights)], out=ym)
                ctx.unmerge(bstate["plan"], ym, a, out=b_)
                ctx.layernorm(b_, *bw2["ln2"], out=xn)
                ctx.mlp(xn, *bw2["mlp"], residual=b_, out=a)

        run_blocks(1)
        ctx.poll()
        barrier()
        ctx.timers_reset()
        ev0.record()
        run_blocks(args.steps)
        ev1.record()
        barrier()
        blk_ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
        ctx.poll()
        bt = ctx.timers_read()
        per = lambda k: round(bt[k][0] / max(bt[k][1], 1), 3)
        block = {"ms_per_block": blk_ms / args.steps, "frames_per_s": aggregate_frames_per_s(wl.frames, args.steps, world, blk_ms),
                 "ms": {"layernorm (x4)": per("layernorm"), "frame_attn": per("frame_attn"), "mlp (x2)": per("mlp"),
                        "merge": per("merge"), "global attention core": per("attention"), "unmerge": per("unmerge")},
                 "note": "one block = frame-local attention + MLP + merged global attention + MLP, pre-norm; "
                         "plan refreshed every %d blocks" % wl.recompute_interval}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (attention core) and per-step breakdown
    att_ms, att_n = timers["attention"]
    att_flops = 4.0 * m * m * d
    att_tflops = att_flops / (att_ms / max(att_n, 1) * 1e-3) / 1e12 if att_ms > 0 else 0.0
    bytes_of = {"merge": (n + m) * d * 2, "unmerge": (m + 2 * n) * d * 2, "var_map": n * d * 2,
                "grad_map": wl.frames * 3 * wl.img_h * wl.img_w * 4}
    flops_of = {"attention": att_flops, "match": 2.0 * ctx.n_src * ctx.n_dst * d, "qkv_proj": 6.0 * m * d * d,
                "out_proj": 2.0 * m * d * d}
    breakdown = {}
    for name, vals in step_samples.items():
        if not vals:
            continue
        med, best = float(np.median(vals)), float(min(vals))
        entry = {"ms_median": round(med, 4), "ms_best": round(best, 4), "samples": len(vals),
                 "ms_x_mhz": round(med * stats_mhz, 1) if stats_mhz else None}
        if name in bytes_of:
            entry["GB/s"] = round(bytes_of[name] / (med * 1e-3) / 1e9, 1)
            entry["frac_hbm"] = round(entry["GB/s"] / peaks["hbm_gbs"], 4)
        if name in flops_of:
            entry["TFLOP/s"] = round(flops_of[name] / (med * 1e-3) / 1e12, 1)
            entry["frac_bf16_sustained"] = round(entry["TFLOP/s"] / peaks["bf16_sustained"], 4)
            entry["frac_bf16_burst"] = round(entry["TFLOP/s"] / peaks["bf16"], 4)
        breakdown[name] = entry

    cpu = run_cpu_baseline(wl, images, tokens, weights[0]) if world == 1 and not args.no_cpu_baseline else None

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": workload_name(wl, n, m),
            "parallelism": "replicas only" if world > 1 else "single GPU",
            "l2": "inputs larger than L2 (x is %.2f GB); no flush between steps" % (n * d * 2 / 1e9),
            "tokens_per_s": world * n * args.steps / (ms / 1e3),
        },
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": n * d * 2, "d2h_bytes_per_step": n * d * 2,
                "ms_per_step": e2e_ms / args.steps,
                "call": "litevggt_global_layer_host_pipelined + litevggt_host_drain: independent steps, pinned "
                        "host buffers, copies on their own streams overlapping the neighbouring steps' kernels"},
        "gpu_launches": launches,
        "roofline": {"kernel": "flash_attention_kernel", "bound": "tensor", "achieved": att_tflops,
                     "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                     "frac": att_tflops / peaks["bf16_sustained"],
                     "frac_of_burst": att_tflops / peaks["bf16"], "peak_burst": peaks["bf16"],
                     "frac_of_nominal_dense": att_tflops / 2250.0,
                     "sm_mhz_median": clocks["sm_mhz"] if clocks else None,
                     "traffic": (ATTENTION_TRAFFIC_C5["bytes_per_layer"]
                                 if wl.name == "C5" and _attention_source_hash() == ATTENTION_TRAFFIC_C5["kernel_sha256"]
                                 else None),
                     "traffic_unit": "bytes per layer (all key-chunk launches of one attention core)",
                     "peak_source": f"{peaks['source']} sustained bf16 (kernel timed inside a long step)",
                     "flops_per_launch": att_flops, "ms_per_launch": att_ms / max(att_n, 1),
                     "launch": "one attention core = the key-chunk launches of one layer, timed as a group"},
        "breakdown": breakdown,
        "breakdown_note": "device time per call from the library's stopwatches over a separate pass of 10 calls per step "
                          "(attention layer: 5 at this size), median and best; ms_x_mhz = median ms x median SM MHz of "
                          "that pass (%s MHz)" % (stats_mhz,),
        "cpu_baseline": cpu,
        "fp8_qkv_variant": fp8,
    }
    if block is not None:
        line["aggregator_block"] = block
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=6)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="C5", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fp8", action="store_true", help="skip the timing of the E4M3 variant of the attention operands")
    ap.add_argument("--block", action="store_true",
                    help="also time whole aggregator blocks (LayerNorm, frame-local attention, MLP around the "
                         "merged global layer) and add an \"aggregator_block\" object to the line")
    ap.add_argument("--interval", type=int, default=None,
                    help="recompute the merge plan every this many layers (default: the workload's, 6); "
                         "with --steps 24 this reproduces the paper's recompute-interval ablation")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    if args.interval is not None:
        if args.interval < 1:
            ap.error("--interval must be >= 1")
        wl = dataclasses.replace(wl, recompute_interval=args.interval)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()

"""Host-side logic of the benchmark: rank aggregation over a 2-process gloo group (the N > 1
path runs independent replicas, so the only cross-rank step is the max over ranks of the timed
region), the extrapolation of the sampled CPU baseline, the clock-sample parser, and the
reference arm's JSON line on the smallest workload."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 100.0 + 50.0 * rank  # rank 1 is the slow replica
    got = bench.max_over_ranks(ms, world, torch.device("cpu"))
    value = bench.aggregate_frames_per_s(1000, 6, world, got)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as fh:
        json.dump({"ms": got, "value": value, "seed": bench.rank_seed(5000, rank)}, fh)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_gloo_replicas_report_the_slowest_rank(tmp_path):
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = json.load(open(tmp_path / "rank0.json"))
    r1 = json.load(open(tmp_path / "rank1.json"))
    assert r0["ms"] == r1["ms"] == 150.0
    # two replicas x 1000 frames x 6 layers in 0.15 s
    assert r0["value"] == pytest.approx(2 * 1000 * 6 / 0.15)
    assert r0["seed"] != r1["seed"]


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks(12.5, 1, torch.device("cpu")) == 12.5
    assert bench.aggregate_frames_per_s(200, 6, 1, 60.0) == pytest.approx(200 * 6 / 0.06)


def test_frames_per_s_amortises_the_plan_over_the_refresh_interval():
    t = dict(grad_map=1.0, var_map=0.2, partition=0.1, index_build=0.1, match=0.5, merge=0.1, qkv_proj=0.2,
             out_proj=0.1, unmerge=0.1, attention=2.0)
    layer = 0.1 + 0.2 + 2.0 + 0.1 + 0.1
    plan = 0.2 + 0.1 + 0.5 + 0.1
    assert bench.frames_per_s_from_steps(t, 160, 6) == pytest.approx(160 / (layer + plan / 6))


def test_oracle_sample_on_c1_scales_row_samples_to_the_whole_problem():
    """The bounded samples of the CPU baseline on config C1, where the samples can cover the whole
    problem: with every src row, every query row and all 16 heads sampled the row-sampled steps are
    the oracle's full calls, so their extrapolation factors are 1."""
    from synthdata import WORKLOADS, make_attention_weights, make_images, make_tokens

    wl = WORKLOADS["C1"]
    images = make_images(wl)
    tokens = make_tokens(wl, images)
    weights = make_attention_weights(wl, 0)
    sample = dict(match_rows=10 ** 6, attn_rows=10 ** 6, attn_heads=16, proj_rows=10 ** 6, linear_frames=wl.frames)
    data = bench.prepare_oracle_sample(wl, images, tokens, weights, sample)
    sz = data["sizes"]
    assert data["match_src"].size == sz["n_src"] and data["match_dst"].size == sz["n_dst"]
    assert data["attn_rows"].size == sz["M"] and len(data["qkv_heads"]) == 16 and data["x_proj"].shape[0] == sz["M"]
    assert data["qkv_heads"][0].shape == (sz["M"], 192)
    t, margin = bench.oracle_sampled_layer(wl, data)
    assert set(t) == {"grad_map", "var_map", "partition", "match", "index_build", "merge", "unmerge", "qkv_proj",
                      "out_proj", "attention"}
    assert all(v > 0 for v in t.values()) and margin.size == sz["n_src"] and np.all(margin >= 0)
    hist = bench.margin_histogram(margin)
    assert 0 <= hist["below_1e-5"] <= hist["below_1e-4"] <= hist["below_1e-3"] <= 1
    # a quarter of the rows sampled: the same call on fewer rows, scaled by rows / sampled rows
    small = bench.prepare_oracle_sample(wl, images, tokens, weights, dict(sample, match_rows=125, attn_rows=136, attn_heads=4))
    assert small["match_src"].size == 125 and small["attn_rows"].size == 136 and len(small["qkv_heads"]) == 4
    assert "125 of 501 src rows" in bench.sample_description(wl, sample, small)


def test_clock_sampler_parses_nvidia_smi_lines():
    s = bench.ClockSampler(0)
    s.proc = type("P", (), {"terminate": lambda self: None, "wait": lambda self, timeout=None: 0})()
    s.lines = ["1965, 1965, 612.2, Not Active, Not Active, Not Active, Not Active",
               "1515, 1965, 998.1, Not Active, Not Active, Not Active, Active",
               "1470, 1965, 1001.0, Not Active, Not Active, Not Active, Active", "garbage"]
    out = s.stop()
    assert out["sm_mhz"] == 1515.0 and out["sm_max_mhz"] == 1965.0 and out["samples"] == 3
    assert out["reasons"] == ["sw_power_cap"]


def test_reference_arm_prints_one_json_line_on_c1():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "C1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "frames/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["config"]["workload"].startswith("C1")

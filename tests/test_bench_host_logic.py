"""Host-side logic of the benchmark: rank aggregation over a 2-process gloo group (the N > 1
path runs independent replicas, so the only cross-rank step is the max over ranks of the timed
region), the extrapolation of the sampled CPU baseline, the clock-sample parser, and the
reference arm's JSON line on the smallest workload."""
import json
import os
import subprocess
import sys

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


def test_extrapolation_scales_quadratic_and_linear_steps():
    t = dict(grad_map=1.0, var_map=0.2, partition=0.1, index_build=0.1, match=0.5, merge=0.1, qkv_proj=0.2,
             out_proj=0.1, unmerge=0.1, attention=2.0)
    # 10x the frames: linear steps x10, quadratic x100; plan amortised over 6 layers
    layer = (0.1 + 0.2 + 0.1 + 0.1) * 10 + 2.0 * 100
    plan = (0.2 + 0.1 + 0.1) * 10 + 0.5 * 100
    assert bench.extrapolate_frames_per_s(t, 16, 160, 6) == pytest.approx(160 / (layer + plan / 6))


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

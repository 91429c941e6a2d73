"""Host-side checks of the benchmark's contract (no GPU): the reference arm (the CPU oracle timed on
a bounded sample) prints one JSON line with the agreed keys, and the committed DRAM-traffic record
that `roofline.traffic` is taken from is consistent with the workloads' algorithmic bytes."""
import json
import os
import subprocess
import sys

from paper_2510_08522_b200 import workload as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                        "--cpu-sample-elems", str(1 << 20)], cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "dmx_step_GBps" and line["unit"] == "GB/s"
    assert line["higher_is_better"] is True and line["vs_baseline"] is None and line["steps"] == 1
    assert line["value"] > 0 and line["ms_per_step"] > 0
    assert line["config"]["workload"] == W.WORKLOADS[4].name
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == line["value"] and cb["sample"]
    assert line["e2e"] == {"value": line["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["gpu_launches"] == 0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_traffic_record_matches_the_algorithmic_bytes():
    """The record holds ncu's DRAM bytes of one launch of the fused kernel per workload (small-case
    captures scaled to full size). Nothing is re-read, so they sit just under the algorithmic
    bytes; in-place state lines that hit L2 take a few per cent off on the small workloads."""
    with open(os.path.join(ROOT, "profiles", "pipe_kernel_dram_traffic.json")) as f:
        rec = json.load(f)
    by_name = {wl.name: wl for wl in W.WORKLOADS}
    assert rec["kernel"] == "dmx::pipe_kernel" and len(rec["kernel_source_digest"]) == 16
    assert {W.WORKLOADS[3].name, W.WORKLOADS[4].name} <= set(rec["traffic_bytes_per_launch"])
    for name, traffic in rec["traffic_bytes_per_launch"].items():
        ratio = traffic / by_name[name].bytes_per_step
        assert 0.9 <= ratio <= 1.02, (name, ratio)

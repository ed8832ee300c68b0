"""The benchmark's reference arm and its accounting helpers, checked on the CPU (no GPU, no CUDA library)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_valid_line():
    """`bench.py --impl reference` times the CPU oracle on the benchmark workload and prints the contract's
    JSON line with impl = reference, zero transfers and its own cpu_baseline description."""
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["higher_is_better"] is False and line["unit"] == "us"
    assert line["value"] > 0 and line["vs_baseline"] is None and line["gpu_launches"] == 0
    assert line["e2e"] == {"value": line["value"], "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == line["value"] and "M=63" in cb["sample"]
    assert "olmoe" in line["config"]["workload"]


def test_reference_arm_other_ranks_exit_quietly():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=120, cwd=ROOT,
                         env=env)
    assert res.returncode == 0 and not [l for l in res.stdout.splitlines() if l.startswith("{")]


def test_algorithmic_bytes_of_the_headline_point():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2602_16052_b200 import synth
    cfg = synth.CONFIGS["olmoe"]
    # 32 kept experts x 3*d*f*2 bytes, plus router, hidden and an fp32 output
    want = 32 * 3 * 2048 * 1024 * 2 + 64 * 2048 * 2 + 63 * 2048 * 2 + 63 * 2048 * 4
    assert bench.algorithmic_bytes(cfg, 63, 32, 4) == want
    assert cfg.expert_weight_bytes() == 3 * 2048 * 1024 * 2


def test_roofline_traffic_comes_from_the_tracked_counters_file():
    """roofline.traffic is read from the counters file kept beside the profiler summary; the file must agree
    with the launches that summary lists and with the algorithmic bytes of the workload."""
    import re
    sys.path.insert(0, ROOT)
    import bench
    from paper_2602_16052_b200 import synth
    c = bench.read_counters()
    assert c is not None, "counters file missing"
    traffic = bench.dram_traffic_per_launch()
    assert traffic == c["dram__bytes_read.sum"] + c["dram__bytes_write.sum"]
    cfg = synth.CONFIGS["olmoe"]
    algo = bench.B_HEADLINE * cfg.expert_weight_bytes()
    assert c["algorithmic_bytes_per_launch"] == algo
    assert 1.0 <= traffic / algo < 1.1, "DRAM traffic should be the weight bytes plus a few per cent"
    # the summary's table rows for the same counters, in MB per captured launch
    md = open(os.path.join(ROOT, "profiles", "ffn_tc_kernel_olmoe_M63_B32.md")).read()
    def row(name):
        m = re.search(r"\| " + re.escape(name) + r" \|([^\n]*)\|", md)
        assert m, name
        return [float(x) for x in re.findall(r"([0-9]+\.[0-9]+) MB", m.group(1))]
    rd, wr = row("dram__bytes_read.sum"), row("dram__bytes_write.sum")
    assert len(rd) == int(c["captured_launches"]) == len(wr)
    assert abs(sum(rd) / len(rd) * 1e6 - c["dram__bytes_read.sum"]) <= 0.01e6 * len(rd) + 1e4
    assert abs(sum(wr) / len(wr) * 1e6 - c["dram__bytes_write.sum"]) <= 0.01e6 * len(wr) + 1e4

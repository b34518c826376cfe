"""The benchmark's reference arm (the CPU oracle timed on a bounded sample) runs without a GPU: one
short invocation must print a single JSON line with the contract's keys, so that the arm cannot break
unseen."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run(*extra):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--reference-budget", "1", *extra],
                         check=True, capture_output=True, text=True, cwd=ROOT, timeout=300).stdout
    lines = [l for l in out.splitlines() if l.strip()]
    assert len(lines) == 1, out
    return json.loads(lines[0])


def test_reference_arm_prints_one_json_line():
    for extra in (("--workload", "cfg1"), ("--workload", "cfg1", "--call", "predict"), ("--workload", "cfg4", "--scale", "small")):
        line = run(*extra)
        assert line["impl"] == "reference" and line["metric"] == "model_cells_per_sec" and line["unit"] == "cells/s"
        assert line["value"] > 0 and line["higher_is_better"] is True and line["gpu_launches"] == 0
        assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
        assert line["cpu_baseline"]["value"] == line["value"] == line["e2e"]["value"]
        assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
        assert line["config"]["workload"].startswith(extra[1])


def test_single_thread_oracle_timing_restores_the_thread_count():
    sys.path.insert(0, ROOT)
    import bench
    from oracle import plogp_oracle as po
    from paper_cs_0408034_b200 import workloads as wl
    n = po.threads()
    v, cores, text = bench.oracle_sample_rate(wl.config1(), 0.2, threads=1)
    assert v > 0 and cores == 1 and po.threads() == n

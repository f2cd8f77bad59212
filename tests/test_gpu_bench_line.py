"""bench.py prints one JSON line with the keys its readers rely on.

Run on the small 4K workload in a process of its own (a few seconds): the line must carry the metric, the timed
region's figures, the roofline of the dominant kernel with its live CUDA-event time behind `achieved`, the same step
as a burst, the end-to-end figure through host buffers with its byte counts, the CPU baseline from the oracle, the
clock record and the launch count, and the figures must be consistent with one another.
"""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*flags):
    res = subprocess.run([sys.executable, "bench.py", "--workload", "gqa4_4k", "--steps", "4", "--warmup", "3", *flags],
                         cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout[-2000:]
    return json.loads(lines[0])


def test_bench_line_carries_the_contract_keys_and_consistent_figures():
    d = run_bench("--no-comparators")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "clocks", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["warmup"] >= 3 and d["higher_is_better"] is True
    assert d["dtype"] == "bf16" and d["data"] == "synthetic" and d["vs_baseline"] is None
    assert d["config"]["workload"] == "gqa4_4k" and "model" not in d["config"]
    assert d["gpu_launches"] > 0
    lat = d["latency_ms"]
    assert lat["kap"] > 0 and lat["osk"] > 0 and abs(lat["kap"] + lat["osk"] - d["ms_per_step"]) < 0.25 * d["ms_per_step"]
    # value = visited-block work over the step time
    blocks = d["config"]["blocks_scored"] + d["config"]["blocks_computed"]
    assert abs(d["value"] - blocks * 2 * 128 ** 3 / (d["ms_per_step"] * 1e-3) / 1e12) < 1e-6 * d["value"] + 1e-9
    r = d["roofline"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert key in r, key
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert 0 < r["frac"] < 1.2
    burst = d["latency_ms_as_a_burst"]
    assert burst["kap"] > 0 and burst["osk"] > 0 and burst["osk"] < 1.5 * lat["osk"]
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and e["value"] < d["value"]
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["value"] > 0 and c["cores"] >= 1 and c["sample"]
    assert "sm_mhz" in d["clocks"] and "reasons" in d["clocks"]


def test_bench_variants_run():
    for flags in (("--block-q", "256", "--osk-impl", "5"), ("--page-size", "16", "--pages-in-place"), ("--top-p", "0.95")):
        d = run_bench("--no-comparators", "--no-cpu-baseline", "--no-e2e", "--no-burst", *flags)
        assert d["value"] > 0 and d["latency_ms"]["osk"] > 0

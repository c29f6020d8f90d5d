"""The benchmark's one-line contract on a real run (small workload): every key the line must carry, the
launch count, the end-to-end leg with host buffers, and the reference arm's line beside it."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                       timeout=900, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout[-2000:]
    return json.loads(lines[0])


def test_our_arm_prints_the_whole_contract():
    d = run_bench("--workload", "tiny_split", "--steps", "4", "--warmup", "3", "--secondary", "tiny",
                  "--secondary-steps", "2")
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert k in d, k
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["warmup"] >= 3 and d["higher_is_better"] is True
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["dtype"] == "bf16" and d["data"] == "synthetic"
    assert d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["config"]["workload"] == "tiny_split" and "model" not in d["config"]
    r = d["roofline"]
    for k in ("bound", "achieved", "peak", "unit", "frac", "traffic", "traffic_source"):
        assert k in r, k
    assert r["bound"] in ("hbm", "tensor", "alu") and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["value"] > 0 and c["cores"] >= 1 and c["sample"]
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < d["value"]                       # the copies are inside its timed region
    # per step: forward, merge, D-prep and the two backward kernels
    assert d["gpu_launches"] == 5 * d["steps"]
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])
    # the second workload of the target, timed after the headline one (here a small stand-in)
    s2 = d["secondary"]
    for k in ("workload", "value", "ms_per_step", "kernel_ms_per_step", "roofline", "bwd_bands", "band_scratch_gb",
              "device_bytes_held", "clocks"):
        assert k in s2, k
    assert s2["workload"] == "tiny" and s2["value"] > 0 and s2["steps"] == 2


def test_reference_arm_prints_its_line():
    d = run_bench("--impl", "reference", "--workload", "tiny", "--steps", "1", "--warmup", "0")
    assert d["impl"] == "reference" and d["dtype"] == "f64" and d["gpu_launches"] == 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0

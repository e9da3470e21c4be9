"""bench.py prints ONE JSON line with the keys the driver reads; checked on a small
workload (the GPU arm) and on a tiny sample (the oracle arm, CPU only)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
             "scaling", "vs_baseline", "dtype", "data", "config", "e2e", "cpu_baseline", "gpu_launches"}


def _run(args, timeout):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT,
                         capture_output=True, text=True, timeout=timeout)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, lines                      # exactly one line on stdout
    return json.loads(lines[0])


def test_reference_arm_prints_the_contract_line():
    line = _run(["--impl", "reference", "--steps", "1", "--warmup", "1", "--cpu-params", "65536"], 600)
    assert BASE_KEYS <= set(line)
    assert line["impl"] == "reference" and line["gpu_launches"] == 0
    assert line["metric"] == "GXPO active-step params/sec" and line["unit"] == "params/s"
    assert line["higher_is_better"] is True and line["vs_baseline"] is None and line["data"] == "synthetic"
    assert line["value"] > 0 and line["steps"] == 1
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["cpu_baseline"]["value"] == line["value"] == line["e2e"]["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert "workload" in line["config"]


@pytest.mark.gpu
def test_gpu_arm_prints_the_contract_line():
    line = _run(["--workload", "flat", "--params", "50000000", "--steps", "3", "--warmup", "3",
                 "--e2e-params", "4194304", "--cpu-params", "65536"], 900)
    assert BASE_KEYS | {"roofline", "clocks", "kernels"} <= set(line)
    assert "impl" not in line or line["impl"] == "ours"
    assert line["metric"] == "GXPO active-step params/sec" and line["unit"] == "params/s"
    assert line["n_gpus"] == 1 and line["steps"] == 3 and line["warmup"] >= 3
    assert line["scaling"] == "weak" and line["dtype"] == "f32" and line["data"] == "synthetic"
    assert line["value"] == pytest.approx(50000000 / (line["ms_per_step"] * 1e-3), rel=1e-9)
    r = line["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0
    assert r["frac"] == pytest.approx(r["achieved"] / r["peak"], rel=1e-12)
    assert r["traffic"] is None or r["traffic"] > 0
    assert r["kernel"] in {k["kernel"] for k in line["kernels"].values()}
    assert 0.3 < r["frac"] < 1.3                        # a real sweep on a real GPU, not a no-op
    assert line["gpu_launches"] == 3 * 4                # three sweeps and the gate kernel per step
    e = line["e2e"]
    assert e["h2d_bytes_per_step"] == 18 * 4194304 and e["d2h_bytes_per_step"] == 12 * 4194304 + 64
    assert 0 < e["value"] < line["value"]               # the host-resident leg is bound by the link
    c = line["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] == 1 and c["value"] > 0
    assert set(line["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert line["config"]["workload"].startswith("flat") and "model" not in line["config"]

"""The JSON line of the benchmark on a GPU: every key of the contract, and numbers that hang together."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_gpu_arm_prints_one_contract_line(cuda_device):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--no-extras", "--steps", "40", "--warmup", "3",
                          "--cpu-seconds", "1"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["metric"] == "ec_allreduce_apply_GBps" and d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 40
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["dtype"] == "f32" and d["data"] == "synthetic" and "workload" in d["config"] and "l2" in d["config"]
    assert d["gpu_launches"] == 3 * 40                                        # three applies per epoch, nothing else
    # value = algorithmic bytes of all steps over the device time of all steps
    step_bytes = d["config"]["algorithmic_bytes_per_step"]
    assert abs(d["value"] - step_bytes / (d["ms_per_step"] * 1e-3) / 1e9) < 0.01 * d["value"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3
    assert 0.5 * step_bytes / 3 < r["traffic"] < 1.2 * step_bytes / 3        # DRAM bytes per launch: near the algorithmic bytes
    assert 3000 < r["achieved"] < 9000                                        # GB/s on a B200
    e = d["e2e"]
    assert e["unit"] == "GB/s" and e["h2d_bytes_per_step"] > 2 ** 30 and e["d2h_bytes_per_step"] >= 2 ** 26
    assert 0 < e["value"] < d["value"] / 10                                   # host buffers: PCIe-bound
    c = d["clocks"]
    assert c["sm_max_mhz"] >= c["sm_mhz"] > 0 and isinstance(c["reasons"], list)
    b = d["cpu_baseline"]
    assert b["kind"] == "oracle" and b["cores"] >= 1 and b["value"] > 0 and b["sample"]

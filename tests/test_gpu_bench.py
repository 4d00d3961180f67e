"""The benchmark's JSON line on a GPU: runs bench.py for a few steps and checks the contract's keys and sanity."""
import json
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent


def test_bench_line_has_the_contract_keys():
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--steps", "5", "--warmup", "3", "--no-cpu-baseline"],
                       cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 5 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["data"] == "synthetic" and "workload" in d["config"] and d["gpu_launches"] == 10
    rf = d["roofline"]
    assert rf["bound"] == "alu" and 0.3 < rf["frac"] < 1.2 and abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9
    assert rf["traffic"] is None or rf["traffic"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 4096 * 4096 * 4 and d["e2e"]["d2h_bytes_per_step"] == 4096 * 4096 * 4
    assert 0 < d["e2e"]["value"] < d["value"]
    assert d["comparison_int8_tensor"].get("int32_result_identical_to_qnn_bgemm", True) is True
    assert abs(d["value"] - 2.0 * 4096 ** 3 * 4 / (d["ms_per_step"] * 1e-3) / 1e12) < 1e-6 * d["value"]

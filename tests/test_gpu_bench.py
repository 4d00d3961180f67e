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
    assert d["e2e"]["result_identical_to_resident_path"] is True
    # every configuration of the workload list is in the same line, each with its own roofline
    c = d["configs"]
    assert "unavailable" not in c, c
    for key in ("config1_fc_64x256x512_w2a2", "config2_conv3x3_256_14x14_b32_w2a2", "config3_gemm_4096",
                "config4_resnet18_b256_w3a3", "config5_vgg16_b64_w4a4", "sweep_8192_bits_1_to_6"):
        assert key in c, key
    assert [(e["wb"], e["ab"]) for e in c["config3_gemm_4096"]] == [(1, 1), (2, 2), (3, 3), (4, 4), (2, 4)]
    assert len(c["config4_resnet18_b256_w3a3"]["layers"]) == 19 and len(c["config5_vgg16_b64_w4a4"]["layers"]) == 13
    assert [e["bits"] for e in c["sweep_8192_bits_1_to_6"]] == [1, 2, 3, 4, 5, 6]
    for e in c["config3_gemm_4096"] + c["sweep_8192_bits_1_to_6"] + [c["config2_conv3x3_256_14x14_b32_w2a2"]]:
        assert e["roofline"]["bound"] == "alu" and 0.2 < e["roofline"]["frac"] < 1.2, e
    for net in ("config4_resnet18_b256_w3a3", "config5_vgg16_b64_w4a4"):
        for L in c[net]["layers"]:
            assert L["roofline"]["bound"] in ("alu", "hbm") and 0.05 < L["roofline"]["frac"] < 1.2, L
    assert abs(c["sweep_8192_bits_1_to_6"][1]["eq16_speedup_model"] - 15.13) < 0.01        # Eq. 16's printed 2-bit value
    # the plain fp32 kernel of the efficiency figure is timed in the same leg; the bit-plane product beats it at every width
    assert c["naive_fp32_8192"]["ms"] > 0
    for e in c["sweep_8192_bits_1_to_6"]:
        assert abs(e["speedup_vs_naive_fp32"] - c["naive_fp32_8192"]["ms"] / e["ms"]) < 1e-9 and e["speedup_vs_naive_fp32"] > 1.0

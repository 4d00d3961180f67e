"""Multi-rank host logic of bench.py on CPU: two gloo ranks (no GPU needed)."""
import json
import socket
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def torchrun(nproc, script_args, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), *script_args]
    return subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=timeout)


def test_two_ranks_agree_on_max_and_shard_rows(tmp_path):
    r = torchrun(2, [str(ROOT / "tests" / "dist_worker.py"), str(tmp_path)])
    assert r.returncode == 0, r.stderr[-2000:]
    d0 = json.loads((tmp_path / "rank0.json").read_text())
    d1 = json.loads((tmp_path / "rank1.json").read_text())
    assert d0["world"] == d1["world"] == 2 and {d0["rank"], d1["rank"]} == {0, 1}
    assert d0["max"] == d1["max"] == [11.0, 5.0]                 # element-wise max over ranks
    assert d0["w_sum"] == d1["w_sum"] and d0["a_sum"] != d1["a_sum"]   # replicated weights, per-rank batches
    one_gpu = 2.0 * 4096 ** 3 * 4 / 2e-3 / 1e12
    assert abs(d0["value"] - 2 * one_gpu) < 1e-6 * one_gpu        # whole-job aggregate: N x per-rank work


def test_reference_arm_prints_one_line_from_rank0_only():
    r = torchrun(2, [str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["unit"] == "binary TOPS" and d["n_gpus"] == 2


def test_cpu_popcount_comparator_leg_reports_all_six_widths():
    """The CPU form of the method timed beside the efficiency sweep: six widths, times that grow with the number of
    plane pairs, and the speed-up against a given GPU sweep computed from the full-size figures."""
    sys.path.insert(0, str(ROOT))
    import bench
    sweep = [{"bits": b, "ms": 2.0 * b * b} for b in range(1, 7)]
    r = bench.cpu_popcount_leg(sweep)
    rows = r["bits_1_to_6"]
    assert [e["bits"] for e in rows] == [1, 2, 3, 4, 5, 6] and r["cores"] >= 1
    assert rows[5]["sample_ms"] > rows[0]["sample_ms"] > 0
    for e in rows:
        assert abs(e["full_size_ms"] - e["sample_ms"] * 256) < 1e-6 * e["full_size_ms"]
        assert abs(e["gpu_speedup"] - e["full_size_ms"] / (2.0 * e["bits"] ** 2)) < 1e-9 * e["gpu_speedup"]

#!/usr/bin/env python
"""Benchmark of the {-1,+1} bit-plane decomposed quantized layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-cpu-baseline]

One step = one pass of the whole hot path over one batch of synthetic input:
qnn_encode_pack (fp32 activations -> bit planes) followed by qnn_bgemm (all plane pairs,
combine, scale) against weights packed offline.  Workload: square GEMM Mg = Ng = Kg = 4096,
2-bit weights x 2-bit activations, A = min(|N(0,1)|, 4), W ~ N(0, 0.02), per-tensor scales.

Prints ONE JSON line (rank 0).  `value` is binary TOPS of the whole step with inputs resident
in HBM; `e2e` is the same metric through qnn_fc_forward_host_pipelined with pinned host buffers
(host<->device copies inside the timed region); `roofline` is for the dominant kernel
(the contraction), timed with CUDA events inside the timed region, against the
bit-operation peak measured by the library's register-resident probe in the same run;
`cpu_baseline` is the CPU oracle timed on the host cores.

With N > 1 (launched by torch.distributed.run) every rank runs the same workload on its own
batch of rows (rows are independent, weights replicated, no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

N_SQ = 4096
AB, WB = 2, 2
NBUF = 4           # rotating input/output sets: 4 x (64 MiB in + 64 MiB out) >> 126 MB of L2
METRIC = "binary TOPS, qnn_encode_pack + qnn_bgemm (equiv. int GOPS and % of roofline alongside)"
UNIT = "binary TOPS"
E2E_CHUNK_ROWS, E2E_STREAMS = 1024, 8   # measured best of a sweep (256..2048 rows, 2..32 streams)
POPC_PER_WORD = 0.5   # popcounts the tiled kernel issues per 32-bit xor word (7:3 bit-column counters)


# DRAM read+write of one qnn_bgemm 4096^3 w2a2 launch (launch 0 of the metrics-only ncu pass whose command
# profiles/bgemm_tiled_4096_w2a2.md lists), valid for the kernel source with this digest only.
NCU_TRAFFIC = {"bytes": 21923584, "kernel_sha256": "332bc1fccf77a343ad6e351743b9655020144b0e992e7a4444c42756e131e323"}


def ncu_traffic_bytes():
    import hashlib
    src = ROOT / "paper_2106_09886_b200" / "csrc" / "bgemm_tiled.cuh"
    if NCU_TRAFFIC["bytes"] is None or not src.exists():
        return None
    digest = hashlib.sha256(src.read_bytes()).hexdigest()
    return NCU_TRAFFIC["bytes"] if digest == NCU_TRAFFIC["kernel_sha256"] else None


def binary_ops(Mg, Ng, Kg, ab, wb):
    return 2.0 * Mg * Ng * Kg * ab * wb


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.1] or [r for (_, r) in self.rows]
        for r in inside:
            parts = [p.strip() for p in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(values, device, use_dist: bool):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if use_dist:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_value(ms_per_step: float, world: int):
    """Binary TOPS of the whole job: every rank processes its own 4096-row batch per step (weak scaling)."""
    return binary_ops(N_SQ, N_SQ, N_SQ, AB, WB) * world / (ms_per_step * 1e-3) / 1e12


def rank_workload(rank: int):
    """Per-rank inputs: the weights are the same on every rank, the activation batch is drawn per rank."""
    from paper_2106_09886_b200 import workloads as wl
    return wl.gemm_config3(0, N_SQ, WB, AB, variant=rank)


# ----------------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle on the host cores
# ----------------------------------------------------------------------------------------------------------

def oracle_step_sample(rows_per_step: int, seed: int = 0):
    """Returns (fn, macs) where fn() runs quantize+FC of `rows_per_step` activation rows against all 4096 columns."""
    import oracle
    from paper_2106_09886_b200 import workloads as wl
    c = wl.gemm_config3(seed, N_SQ, WB, AB)
    sa, sw = wl.per_tensor_scale(c.a, AB), wl.per_tensor_scale(c.w, WB)
    alpha = np.float32(sa * sw)
    qw = oracle.quantize(c.w, WB, sw)          # offline, like the packed weights of the GPU arm
    a = c.a

    def fn(step: int):
        r0 = (step * rows_per_step) % (N_SQ - rows_per_step + 1)
        qa = oracle.quantize(a[r0:r0 + rows_per_step], AB, sa)
        acc = oracle.fc(qa, qw)
        return oracle.scale(acc, alpha)

    return fn, oracle.num_threads()


def run_reference(args):
    rank, world, _ = dist_setup(args.gpus)
    if rank != 0:
        return
    rows = 256
    fn, cores = oracle_step_sample(rows)
    for s in range(args.warmup):
        fn(s)
    t0 = time.perf_counter()
    for s in range(args.steps):
        fn(s)
    dt = (time.perf_counter() - t0) / args.steps
    value = binary_ops(rows, N_SQ, N_SQ, AB, WB) / dt / 1e12
    sample = f"{rows} of {N_SQ} activation rows per step (quantize + naive int FC against all {N_SQ} columns + scale)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": f"qnn_bgemm {N_SQ}x{N_SQ}x{N_SQ} w{WB}a{AB} (square GEMM sweep, 2x2 bits)", "sample": sample},
        "equiv_int_gops": 2.0 * rows * N_SQ * N_SQ / dt / 1e9,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------------------------------------

def measure_peaks(torch, qnn, dev):
    """In-run peaks: bit-operation probes (both instruction mixes) and a plain device copy."""
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    sink = torch.empty(sms * 8 * 256, dtype=torch.int32, device=dev)
    res = {}
    for variant, name, iters in ((0, "xor_popc_add", 4000), (1, "csa_3to2", 4000), (2, "kernel_mix_smem", 100),
                                 (3, "mma_sync_b1_and_popc", 500), (4, "mma_sync_b1_xor_popc", 500)):
        best = 0.0
        for _ in range(4):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ops = qnn.probe_bitops(variant, iters, sms * 8, sink)
            e1.record()
            e1.synchronize()
            best = max(best, ops / (e0.elapsed_time(e1) * 1e-3))
        res[name] = best * 64.0 / 1e12            # word-ops/s -> binary TOPS (32 MACs x 2 ops per word)
    nbytes = 1 << 30
    src = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    dst = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    src.zero_()
    best = 0.0
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        qnn.probe_copy(dst, src)
        e1.record()
        e1.synchronize()
        best = max(best, 2.0 * nbytes / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    res["copy_gbs"] = best
    del src, dst
    return res


def int8_tensor_comparison(torch, qnn, dev, a_dev, w_host, sa, sw, planes, packed, alpha):
    """Comparison only: the same integer product computed as ONE int8 tensor-core GEMM on the unpacked odd
    codes (library call: cuBLASLt through torch._int_mm), i.e. what the binary decomposition competes with
    on this GPU.  The codes are rebuilt from the library's own bit planes, and the int32 result is checked
    to be identical to qnn_bgemm's accumulators."""
    try:
        Mg, Kg = a_dev.shape
        def codes_from_planes(pl, bits, k):
            # pl: int32 [rows, bits, kw]; q = 2t - (2^bits - 1), bit i of t = plane i
            rows = pl.shape[0]
            shifts = torch.arange(32, device=dev, dtype=torch.int32)
            t = torch.zeros((rows, pl.shape[2] * 32), dtype=torch.int32, device=dev)
            for i in range(bits):
                bitsv = (pl[:, i, :].unsqueeze(-1) >> shifts) & 1
                t += bitsv.reshape(rows, -1) << i
            return (2 * t[:, :k] - (2 ** bits - 1)).to(torch.int8).contiguous()
        wp, _ = qnn.weights_views(packed, N_SQ, 1, N_SQ, WB)
        qa = codes_from_planes(planes, AB, Kg)
        qw = codes_from_planes(wp, WB, Kg)
        qwt = qw.t().contiguous().t()          # column-major operand, as cuBLASLt's int8 path wants
        ref = torch._int_mm(qa, qw.t())
        _, acc = qnn.bgemm(planes, AB, packed, WB, Mg, N_SQ, Kg, alpha, want_acc=True)
        torch.cuda.synchronize()
        same = bool(torch.equal(ref, acc))
        for _ in range(3):
            torch._int_mm(qa, qw.t())
        torch.cuda.synchronize()
        times = []
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch._int_mm(qa, qw.t())
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = statistics.median(times)
        # the same product through this library's own tcgen05 kind::i8 kernel (unpack of both operands included)
        ws = torch.empty(qnn.lib.qnn_bgemm_int8_tensor_workspace(Mg, N_SQ, Kg), dtype=torch.uint8, device=dev)
        out8 = torch.empty((Mg, N_SQ), dtype=torch.float32, device=dev)
        acc8 = torch.empty((Mg, N_SQ), dtype=torch.int32, device=dev)
        qnn.bgemm_int8_tensor(planes, AB, packed, WB, Mg, N_SQ, Kg, alpha, out=out8, acc=acc8, workspace=ws)
        torch.cuda.synchronize()
        same8 = bool(torch.equal(acc8, acc))
        own = []
        for _ in range(13):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            qnn.bgemm_int8_tensor(planes, AB, packed, WB, Mg, N_SQ, Kg, alpha, want_acc=False, out=out8, workspace=ws)
            e1.record()
            e1.synchronize()
            own.append(e0.elapsed_time(e1))
        ms8 = statistics.median(own[3:])
        return {"what": "int8 tensor-core GEMM on the unpacked odd codes, cuBLASLt via torch._int_mm (library call, comparison only)",
                "ms": ms, "equiv_int_gops": 2.0 * Mg * N_SQ * Kg / (ms * 1e-3) / 1e9, "int32_result_identical_to_qnn_bgemm": same,
                "own_tcgen05_i8": {"what": "qnn_bgemm_int8_tensor: planes -> int8 codes (both operands) + tcgen05 kind::i8 GEMM, fp32 output (comparison only)",
                                   "ms": ms8, "equiv_int_gops": 2.0 * Mg * N_SQ * Kg / (ms8 * 1e-3) / 1e9,
                                   "int32_result_identical_to_qnn_bgemm": same8,
                                   "tensor_path_status": qnn.tensor_path_status()}}
    except Exception as exc:   # comparison only: never fail the benchmark over it
        return {"what": "int8 tensor-core GEMM comparison", "unavailable": f"{type(exc).__name__}: {exc}"[:200]}


def training_side_leg(torch, qnn, dev, planes, packed, mp, mp_kind):
    """Outside the timed step: the backward products of the same layer (Algorithm 1 backward) as TF32 tensor-core
    GEMMs and the streaming encoder derivative, with CUDA events, against the measured bf16 peak scaled by the
    nominal TF32:bf16 ratio and the measured copy peak."""
    try:
        wp, _ = qnn.weights_views(packed, N_SQ, 1, N_SQ, WB)
        wp = wp.contiguous()
        m = n = k = N_SQ
        gen = torch.Generator(device=dev).manual_seed(7)
        grads = [torch.randn((m, n), device=dev, generator=gen) for _ in range(2)]
        x = torch.rand((m, k), device=dev, generator=gen) * 2 - 1
        outs = [torch.empty((m, k), dtype=torch.float32, device=dev) for _ in range(2)]
        gws = [torch.empty((n, k), dtype=torch.float32, device=dev) for _ in range(2)]
        wsd = torch.empty(qnn.lib.qnn_bgemm_backward_data_workspace(m, n, k), dtype=torch.uint8, device=dev)
        wsw = torch.empty(qnn.lib.qnn_bgemm_backward_weights_workspace(m, n, k), dtype=torch.uint8, device=dev)
        alpha = 1.0 / ((2 ** AB - 1) * (2 ** WB - 1))

        def timed(fn, reps=20):
            for i in range(3):
                fn(i)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(reps):
                fn(i)
            e1.record()
            e1.synchronize()
            return e0.elapsed_time(e1) / reps

        t_data = timed(lambda i: qnn.bgemm_backward_data(grads[i % 2], wp, k, WB, alpha, out=outs[i % 2], workspace=wsd))
        t_enc = timed(lambda i: qnn.bgemm_backward_data(grads[i % 2], wp, k, WB, alpha, x=x, ab=AB, r=1.0, out=outs[i % 2],
                                                        workspace=wsd))
        t_w = timed(lambda i: qnn.bgemm_backward_weights(grads[i % 2], planes, k, AB, alpha, gw=gws[i % 2], workspace=wsw))
        gc = torch.randn((AB, m * k), device=dev, generator=gen)
        gx = torch.empty(m * k, dtype=torch.float32, device=dev)
        t_mb = timed(lambda i: qnn.mbit_encoder_backward(x.view(-1), gc, AB, 1.0, gx=gx))
        status = qnn.tensor_path_status()
        flop = 2.0 * m * n * k
        peak = mp["bf16_tflops"] * (1.1 / 2.25)
        # the same for convolution layers: the single-convolution configuration's layer and a mid-sized one
        from paper_2106_09886_b200 import run_case as rc
        conv = []
        for (cn, ch, cc, cco) in ((32, 14, 256, 256), (16, 56, 256, 256)):
            r = rc.time_backward_conv(cn, ch, ch, cc, cco, 3, 3, 1, 1, AB, WB, reps=10, warmup=3)
            conv.append({"layer": f"conv3x3 {cc}->{cco}, {ch}x{ch}, batch {cn}, stride 1, pad 1", "data_ms": r["data_ms"],
                         "weights_ms": r["weights_ms"], "data_tflops": r["data_tflops"], "weights_tflops": r["weights_tflops"],
                         "data_frac_of_tf32_peak": r["data_tflops"] / peak, "weights_frac_of_tf32_peak": r["weights_tflops"] / peak,
                         "workspace_mb": r["workspace_mb"], "tensor_path_status": r["status"]})
        return {"what": "Algorithm 1 backward of the benchmarked layer: whole calls (code unpack / transpose + TF32 tcgen05 GEMM), CUDA events",
                "workload": f"fc {m}x{n}x{k}, w{WB}a{AB}", "dtype": "tf32 x exact codes, fp32 accumulate",
                "backward_data_ms": t_data, "backward_data_with_encoder_derivative_ms": t_enc, "backward_weights_ms": t_w,
                "backward_data_tflops": flop / (t_data * 1e-3) / 1e12, "backward_weights_tflops": flop / (t_w * 1e-3) / 1e12,
                "roofline": {"bound": "tensor", "achieved": flop / (t_data * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                             "frac": flop / (t_data * 1e-3) / 1e12 / peak,
                             "peak_kind": f"{mp_kind} bf16 burst x 1.1/2.25 (nominal TF32:bf16)"},
                "mbit_encoder_backward_gbs": m * k * 4.0 * (2 + AB) / (t_mb * 1e-3) / 1e9, "tensor_path_status": status,
                "convolution_backward": conv}
    except Exception as exc:   # reported beside the benchmark, never fails it
        return {"what": "Algorithm 1 backward", "unavailable": f"{type(exc).__name__}: {exc}"[:200]}


def eq16_model_speedup(n: int, m_bits: int, k_bits: int, gamma: float = 1.91, reg_len: int = 64) -> float:
    """The paper's cost model of its efficiency experiment (Eq. 16): n multiply-accumulates worth gamma bit
    operations each, against M*K plane pairs of gamma + 2*ceil(n/L) operations plus M*K - 1 combining additions
    of beta = gamma/2 each."""
    pairs = m_bits * k_bits
    return n * gamma / (pairs * (gamma + 2 * ((n + reg_len - 1) // reg_len)) + (pairs - 1) * gamma / 2.0)


def configs_leg(torch, qnn, dev, peaks, mp, mp_kind, quick=False):
    """Outside the timed step: every configuration of the workload list, each call timed alone with CUDA events.
    Configurations 1-3 run on the seeded host-generated tensors (L2 flushed before every timed call; the two small
    ones also warm), the two convolution stacks and the 8192^3 sweep on device-drawn tensors of the stated shapes
    and distributions (their outputs are larger than L2).  Every entry carries its own roofline: the slower of its
    algorithmic bytes at the measured HBM peak and its popcount instructions at this run's popcount rate."""
    import statistics as st
    from paper_2106_09886_b200 import run_case as rc
    from paper_2106_09886_b200 import workloads as wl
    popc_per_s = peaks["xor_popc_add"] * 1e12 / 64.0          # the plain probe issues one popcount per word operation
    hbm = mp["hbm_gbs"]
    reps = 3 if quick else 7
    med = lambda f, flush=True, n=reps: st.median(rc._time_calls(f, n, 3, flush=flush))

    def entry(Mg, Ng, Kg, ab, wb, ms, roof, extra=None):
        e = {"Mg": Mg, "Ng": Ng, "Kg": Kg, "ab": ab, "wb": wb, "ms": ms,
             "binary_tops": binary_ops(Mg, Ng, Kg, ab, wb) / (ms * 1e-3) / 1e12,
             "equiv_int_gops": 2.0 * Mg * Ng * Kg / (ms * 1e-3) / 1e9, "roofline": roof}
        if extra:
            e.update(extra)
        return e

    def fc_case(a, w, k_major, ab, wb, warm_too):
        Mg, Kg = a.shape
        Ng = w.shape[1] if k_major else w.shape[0]
        sa, sw = wl.per_tensor_scale(a, ab), wl.per_tensor_scale(w, wb)
        alpha = float(np.float32(sa * sw))
        a_d = torch.from_numpy(a).to(dev)
        packed = qnn.pack_weights(torch.from_numpy(np.ascontiguousarray(w)).to(dev), Ng, 1, Kg,
                                  qnn.W_TCN if k_major else qnn.W_NTC, wb, sw)
        planes = torch.empty((Mg, ab, qnn.row_words(Kg)), dtype=torch.int32, device=dev)
        out = torch.empty((Mg, Ng), dtype=torch.float32, device=dev)
        enc = lambda i: qnn.encode_pack(a_d, ab, sa, 0, planes=planes)
        gemm = lambda i: qnn.bgemm(planes, ab, packed, wb, Mg, Ng, Kg, alpha, out=out)
        enc(0)
        t_enc, t = med(enc), med(gemm)
        extra = {"encode_ms": t_enc, "l2": "flushed before every timed call"}
        if warm_too:
            extra["ms_warm"], extra["encode_ms_warm"] = med(gemm, flush=False), med(enc, flush=False)
        return entry(Mg, Ng, Kg, ab, wb, t, rc.layer_roofline(Mg, Ng, ab, wb, False, 1, 1, Kg, Mg, t, popc_per_s, hbm), extra)

    res = {"method": "CUDA events around single calls, median of %d after 3 warm-up calls; roofline per entry = "
                     "max(algorithmic bytes / measured HBM peak, popcounts / popcount rate of this run's probe)" % reps,
           "popcount_rate_gpops": popc_per_s / 1e9, "hbm_peak_gbs": hbm, "hbm_peak_kind": mp_kind}
    c1 = wl.fc_config1(0)
    res["config1_fc_64x256x512_w2a2"] = fc_case(c1.a, c1.w, c1.k_major, c1.ab, c1.wb, True)
    res["config1_fc_64x256x512_w2a2"]["note"] = "launch-latency-bound: 33.6 M binary MACs; the roofline fraction only says so"

    c2 = wl.conv_config2(0)
    s2 = c2.shape
    sa, sw = wl.per_tensor_scale(c2.a, s2.ab), wl.per_tensor_scale(c2.w, s2.wb)
    alpha = float(np.float32(sa * sw))
    a_d = torch.from_numpy(c2.a).to(dev).view(-1, s2.C)
    packed = qnn.pack_weights(torch.from_numpy(c2.w).to(dev), s2.Cout, 9, s2.C, qnn.W_NTC, s2.wb, sw)
    planes = torch.empty((a_d.shape[0], s2.ab, qnn.row_words(s2.C)), dtype=torch.int32, device=dev)
    out = torch.empty((s2.N, s2.Ho, s2.Wo, s2.Cout), dtype=torch.float32, device=dev)
    enc = lambda i: qnn.encode_pack(a_d, s2.ab, sa, 0, planes=planes)
    conv = lambda i: qnn.bconv2d(planes, s2.ab, packed, s2.wb, s2.N, s2.H, s2.W, s2.C, s2.Cout, 3, 3, 1, 1, alpha, out=out)
    enc(0)
    t_enc, t = med(enc), med(conv)
    res["config2_conv3x3_256_14x14_b32_w2a2"] = entry(
        s2.Mg, s2.Cout, s2.Kg, s2.ab, s2.wb, t,
        rc.layer_roofline(s2.Mg, s2.Cout, s2.ab, s2.wb, True, 3, 3, s2.C, s2.N * s2.H * s2.W, t, popc_per_s, hbm),
        {"encode_ms": t_enc, "ms_warm": med(conv, flush=False), "encode_ms_warm": med(enc, flush=False),
         "l2": "flushed before every timed call (ms), not flushed (ms_warm)"})
    del a_d, packed, planes, out

    c3 = wl.gemm_config3(0, N_SQ, 2, 2)
    res["config3_gemm_4096"] = []
    for wb, ab in wl.GEMM_SWEEP_BITS:
        e = fc_case(c3.a, c3.w, False, ab, wb, False)
        res["config3_gemm_4096"].append(e)

    for key, net, batch in (("config4_resnet18_b256_w3a3", "resnet18", 256), ("config5_vgg16_b64_w4a4", "vgg16", 64)):
        r = rc.time_stack(net, batch, reps=3, warmup=2)
        layers, roof_ms = [], 0.0
        for L in r["layers"]:
            roof = rc.layer_roofline(L["Mg"], L["Ng"], L["ab"], L["wb"], True, L["R"], L["S"], L["C"], L["in_rows"],
                                     L["conv_ms"], popc_per_s, hbm)
            roof_ms += roof["roofline_ms"]
            layers.append({"layer": L["layer"], "Mg": L["Mg"], "Ng": L["Ng"], "Kg": L["Kg"], "encode_ms": L["encode_ms"],
                           "conv_ms": L["conv_ms"], "conv_encode_fused_ms": L["conv_encode_ms"],
                           "binary_tops": L["conv_binary_tops"], "equiv_int_gops": L["conv_equiv_int_gops"],
                           "encode_gbs": L["encode_gbs"],
                           "roofline": {k: roof[k] for k in ("bound", "achieved", "peak", "unit", "frac")}})
        conv_ms = sum(L["conv_ms"] for L in r["layers"])
        res[key] = {"batch": batch, "layers": layers, "total_ms": r["total_ms"], "conv_ms": conv_ms,
                    "encode_ms": r["total_ms"] - conv_ms,
                    "chained_fused_ms": sum(L["conv_encode_ms"] for L in r["layers"]),
                    "binary_tops": r["binary_tops"], "equiv_int_gops": r["equiv_int_gops"],
                    "roofline": {"bound": "alu (per layer: see layers)", "frac": roof_ms / conv_ms,
                                 "what": "sum of the layers' roofline times / sum of their measured convolution times"}}

    # the paper's efficiency experiment (Section 5.4, Fig. 7): 8192^3, 1..6 bits, set against the plain
    # one-thread-per-output fp32 kernel of the same size and against the Eq. 16 cost model
    sweep, base = [], None
    n8 = 8192
    fa = torch.randn(n8, n8, device="cuda")
    fb = torch.randn(n8, n8, device="cuda")
    fc = torch.empty(n8, n8, device="cuda")
    naive_ms = st.median(rc._time_calls(lambda i: qnn.probe_naive_sgemm(fa, fb, fc), 2, 1))
    del fa, fb, fc
    res["naive_fp32_8192"] = {"what": "qnn_probe_naive_sgemm: one thread per output, one fma per step, no tiling "
                                      "(the comparison line of the paper's efficiency figure; not a product path)",
                              "ms": naive_ms, "tflops": 2.0 * n8 ** 3 / naive_ms / 1e9}
    for b in range(1, 7):
        r = rc.time_gemm(n8, n8, n8, b, b, reps=3, warmup=2, sets=1)
        ms = r["ms_median"]
        base = base or ms
        roof = rc.layer_roofline(n8, n8, b, b, False, 1, 1, n8, n8, ms, popc_per_s, hbm)
        sweep.append({"bits": b, "ms": ms, "binary_tops": r["binary_tops"], "equiv_int_gops": r["equiv_int_gops"],
                      "time_vs_1bit": ms / base, "eq16_cost_vs_1bit": eq16_model_speedup(n8, 1, 1) / eq16_model_speedup(n8, b, b),
                      "eq16_speedup_model": eq16_model_speedup(n8, b, b),
                      "speedup_vs_naive_fp32": naive_ms / ms,
                      "roofline": {k: roof[k] for k in ("bound", "achieved", "peak", "unit", "frac")}})
    res["sweep_8192_bits_1_to_6"] = sweep
    return res


def load_measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return json.loads(p.read_text()), "measured"
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


def cpu_baseline_leg():
    rows = 1024
    fn, cores = oracle_step_sample(rows)
    fn(0)
    t0 = time.perf_counter()
    reps = 0
    while True:
        fn(reps)
        reps += 1
        if time.perf_counter() - t0 > 10.0 or reps >= 8:
            break
    dt = (time.perf_counter() - t0) / reps
    return {"value": binary_ops(rows, N_SQ, N_SQ, AB, WB) / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{rows} of {N_SQ} activation rows (quantize + naive int FC against all {N_SQ} columns + scale), "
                      f"{reps} repetitions, {dt:.2f} s each",
            "equiv_int_gops": 2.0 * rows * N_SQ * N_SQ / dt / 1e9}


def cpu_popcount_leg(sweep):
    """The method's own CPU form beside the efficiency sweep (Section 5.4): Eq. 8 on packed planes as the oracle
    writes it (plain C, the compiler's popcount builtin, OpenMP over rows; nothing vectorised by hand), timed on a
    bounded sample of the 8192^3 product for 1..6 bits."""
    import oracle
    n8, rows = 8192, 32
    kw = oracle.row_words(n8)
    rng = np.random.default_rng(8192)
    out = []
    for b in range(1, 7):
        pa = rng.integers(0, 2 ** 32, size=(rows, b, kw), dtype=np.uint64).astype(np.uint32)
        pw = rng.integers(0, 2 ** 32, size=(n8, b, kw), dtype=np.uint64).astype(np.uint32)
        oracle.fc_bitplanes(pa[:2], pw, n8)
        t0 = time.perf_counter()
        oracle.fc_bitplanes(pa, pw, n8)
        dt = time.perf_counter() - t0
        e = {"bits": b, "sample_ms": dt * 1e3, "binary_tops": binary_ops(rows, n8, n8, b, b) / dt / 1e12,
             "full_size_ms": dt * 1e3 * n8 / rows}
        gpu = next((s for s in sweep if s.get("bits") == b), None) if sweep else None
        if gpu:
            e["gpu_speedup"] = e["full_size_ms"] / gpu["ms"]
        out.append(e)
    return {"what": "oracle.fc_bitplanes (Eq. 8 with xor + popcount on packed planes, plain C, OpenMP over rows)",
            "cores": oracle.num_threads(), "sample": f"{rows} of {n8} rows against all {n8} columns, K = {n8}, one call per width",
            "bits_1_to_6": out}


def run_gpu(args):
    import torch
    from paper_2106_09886_b200 import build as lib_build
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        lib_build.build()          # no-op when the library on disk matches the sources
    from paper_2106_09886_b200 import qnn
    from paper_2106_09886_b200 import workloads as wl

    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # ---- workload: per-rank batch of rows (seeded per rank), replicated weights, packed offline
    c = rank_workload(rank)
    sa, sw = wl.per_tensor_scale(c.a, AB), wl.per_tensor_scale(c.w, WB)
    alpha = float(np.float32(sa * sw))
    Mg = Ng = Kg = N_SQ
    w_d = torch.from_numpy(c.w).to(dev)
    packed = qnn.pack_weights(w_d, Ng, 1, Kg, qnn.W_NTC, WB, sw)
    del w_d
    a_host = torch.from_numpy(c.a).pin_memory()
    a_bufs = [a_host.to(dev) for _ in range(NBUF)]
    out_bufs = [torch.empty((Mg, Ng), dtype=torch.float32, device=dev) for _ in range(NBUF)]
    planes = [torch.empty((Mg, AB, qnn.row_words(Kg)), dtype=torch.int32, device=dev) for _ in range(NBUF)]
    out_host = torch.empty((Mg, Ng), dtype=torch.float32).pin_memory()
    torch.cuda.synchronize()

    def step(i):
        b = i % NBUF
        qnn.encode_pack(a_bufs[b], AB, sa, 0, planes=planes[b])
        qnn.bgemm(planes[b], AB, packed, WB, Mg, Ng, Kg, alpha, out=out_bufs[b])

    def barrier():
        torch.cuda.synchronize()
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = measure_peaks(torch, qnn, dev) if rank == 0 else None
    comparison = None
    if rank == 0 and world == 1:
        qnn.encode_pack(a_bufs[0], AB, sa, 0, planes=planes[0])
        comparison = int8_tensor_comparison(torch, qnn, dev, a_bufs[0], c.w, sa, sw, planes[0], packed, alpha)

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.25)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    t_wall0 = time.time()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for i in range(args.steps):
        b = i % NBUF
        ev[i][0].record()
        qnn.encode_pack(a_bufs[b], AB, sa, 0, planes=planes[b])
        ev[i][1].record()
        qnn.bgemm(planes[b], AB, packed, WB, Mg, Ng, Kg, alpha, out=out_bufs[b])
        ev[i][2].record()
    stop.record()
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    ms_total = start.elapsed_time(stop)
    enc_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    gemm_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)

    # ---- end to end through the host-buffer entry point
    e2e_streams = [torch.cuda.Stream(device=dev) for _ in range(args.e2e_streams)]

    def e2e_step(i, last=True):
        # consecutive steps pipeline into each other on the same streams (step i+1's copies in overlap step i's
        # kernels and copies out); the last step of a batch joins the streams before the closing event
        b = i % NBUF
        qnn.fc_forward_host_pipelined(a_host, AB, sa, 0, packed, WB, Ng, alpha, out_host, a_bufs[b], planes[b],
                                      out_bufs[b], args.e2e_chunk_rows, e2e_streams, join=last)

    e2e_steps = max(3, min(args.steps, 50))
    for i in range(3):
        e2e_step(i)
    barrier()
    s2, t2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    for i in range(e2e_steps):
        e2e_step(i, last=(i == e2e_steps - 1))
    t2.record()
    barrier()
    e2e_ms_total = s2.elapsed_time(t2)
    # the end-to-end result, all of it, against the plain two-call route on the resident copy of the same input
    ref_planes = qnn.encode_pack(a_bufs[0], AB, sa, 0)
    ref_out = qnn.bgemm(ref_planes, AB, packed, WB, Mg, Ng, Kg, alpha)
    torch.cuda.synchronize()
    e2e_identical = bool(torch.equal(ref_out.cpu(), out_host))
    del ref_planes, ref_out

    ms_total, e2e_ms_total = max_over_ranks([ms_total, e2e_ms_total], dev, use_dist)

    if rank == 0:
        ms_step = ms_total / args.steps
        ops_step = binary_ops(Mg, Ng, Kg, AB, WB) * world
        value = whole_job_value(ms_step, world)
        e2e_ms = e2e_ms_total / e2e_steps
        mp, mp_kind = load_measured_peaks()
        # The plain probe is popcount-issue bound (one popcount per word), so it measures the popcount
        # pipe; the kernel's 7:3 carry-save mix needs 4 popcounts per 8 words.
        kernel_peak = peaks["xor_popc_add"] / POPC_PER_WORD
        sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
        peak_analytic = 16.0 / POPC_PER_WORD * 148 * sm_mhz * 1e6 * 64.0 / 1e12
        achieved = binary_ops(Mg, Ng, Kg, AB, WB) / (gemm_ms * 1e-3) / 1e12
        alg_bytes_gemm = Mg * Kg * AB / 8 + Ng * Kg * WB / 8 + Mg * Ng * 4
        enc_bytes = Mg * Kg * 4 + Mg * Kg * AB / 8
        traffic = ncu_traffic_bytes()
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int32", "data": "synthetic",
            "config": {"workload": f"qnn_bgemm {N_SQ}x{N_SQ}x{N_SQ} w{WB}a{AB} per GPU (square GEMM sweep, 2x2 bits), "
                                   "step = qnn_encode_pack + qnn_bgemm, weights packed offline",
                       "l2": f"{NBUF} rotating input/output sets of 128 MiB each (larger than L2)",
                       "parallelism": f"replicas x{world}, rows sharded, no collective"},
            "equiv_int_gops": 2.0 * Mg * Ng * Kg * world / (ms_step * 1e-3) / 1e9,
            "kernel_ms": {"qnn_encode_pack": enc_ms, "qnn_bgemm": gemm_ms},
            "gpu_launches": 2 * args.steps,
            "e2e": {"value": ops_step / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": Mg * Kg * 4, "d2h_bytes_per_step": Mg * Ng * 4, "steps": e2e_steps,
                    "api": f"qnn_fc_forward_host_pipelined (pinned host buffers, {args.e2e_chunk_rows}-row chunks over "
                           f"{args.e2e_streams} streams, consecutive steps pipelined)",
                    "result_identical_to_resident_path": e2e_identical},
            "roofline": {"kernel": "qnn_bgemm", "bound": "alu", "achieved": achieved, "peak": kernel_peak,
                         "unit": UNIT, "frac": achieved / kernel_peak, "traffic": traffic,
                         "peak_source": "popcount issue rate measured in this run by the register-resident xor+popc+add "
                                        "probe (popcount-bound, 1 per word), divided by the kernel's 0.5 popcounts per "
                                        "word (of measured)",
                         "peak_analytic": peak_analytic,
                         "probe_xor_popc_add": peaks["xor_popc_add"], "probe_csa_3to2": peaks["csa_3to2"],
                         "probe_kernel_mix_smem": peaks["kernel_mix_smem"],
                         "probe_mma_sync_b1_and_popc": peaks["mma_sync_b1_and_popc"],
                         "probe_mma_sync_b1_xor_popc": peaks["mma_sync_b1_xor_popc"],
                         "frac_of_kernel_mix_probe": achieved / peaks["kernel_mix_smem"],
                         "algorithmic_bytes": alg_bytes_gemm,
                         "hbm_time_ms": alg_bytes_gemm / (mp["hbm_gbs"] * 1e9) * 1e3,
                         "hbm_peak_gbs": mp["hbm_gbs"], "hbm_peak_kind": mp_kind, "copy_probe_gbs": peaks["copy_gbs"]},
            "roofline_encode": {"kernel": "qnn_encode_pack", "bound": "hbm", "achieved": enc_bytes / (enc_ms * 1e-3) / 1e9,
                                "peak": mp["hbm_gbs"], "unit": "GB/s",
                                "frac": enc_bytes / (enc_ms * 1e-3) / 1e9 / mp["hbm_gbs"], "peak_kind": mp_kind},
            "clocks": clocks,
        }
        if comparison is not None:
            line["comparison_int8_tensor"] = comparison
        if world == 1:
            line["training_side"] = training_side_leg(torch, qnn, dev, planes[0], packed, mp, mp_kind)
        if world == 1 and not args.no_configs:
            sampler2 = ClockSampler(local)                # the per-configuration table runs for seconds: its own clock record
            sampler2.start()
            t_c0 = time.time()
            try:
                line["configs"] = configs_leg(torch, qnn, dev, peaks, mp, mp_kind)
            except Exception as exc:   # reported beside the benchmark, never fails it
                line["configs"] = {"unavailable": f"{type(exc).__name__}: {exc}"[:300]}
            line["configs"]["clocks"] = sampler2.stop(t_c0, time.time())
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_leg()
            sweep = line.get("configs", {}).get("sweep_8192_bits_1_to_6") if isinstance(line.get("configs"), dict) else None
            line["cpu_popcount_8192"] = cpu_popcount_leg(sweep)
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["graft", "reference"], default="graft")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration table (configs 1-5 and the 8192^3 sweep)")
    ap.add_argument("--e2e-chunk-rows", type=int, default=E2E_CHUNK_ROWS, help="rows per chunk of the end-to-end pipeline")
    ap.add_argument("--e2e-streams", type=int, default=E2E_STREAMS, help="streams of the end-to-end pipeline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.impl == "reference":
        run_reference(args)
    else:
        if args.warmup < 3:
            args.warmup = 3
        run_gpu(args)


if __name__ == "__main__":
    main()

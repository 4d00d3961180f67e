"""Run one library call on synthetic device data a few times and print its timing (one JSON line).

    python -m paper_2106_09886_b200.run_case gemm   --m 4096 --n 4096 --k 4096 --ab 2 --wb 2 [--reps 5]
    python -m paper_2106_09886_b200.run_case conv   --N 32 --H 14 --W 14 --C 256 --Cout 256 --R 3 --S 3 --stride 1 --pad 1 --ab 2 --wb 2
    python -m paper_2106_09886_b200.run_case encode --rows 4096 --k 4096 --bits 2
    python -m paper_2106_09886_b200.run_case backward_conv --N 32 --H 14 --W 14 --C 256 --Cout 256
    python -m paper_2106_09886_b200.run_case stack  --net vgg16 [--batch 64] [--layers 0,1] [--table]

Inputs are drawn on the device (half-normal activations, normal weights); this is a timing and
profiling driver, correctness is the business of the test-suite.  Times are CUDA-event times of
the single library call, after `--warmup` untimed calls, rotating over `--sets` input/output sets
so that consecutive calls do not find their data in L2.
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

from . import qnn


_flush_buf = None


def flush_l2():
    """Writes a buffer twice the size of the L2 cache, so that the next call finds none of its data there."""
    global _flush_buf
    if _flush_buf is None:
        _flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    _flush_buf.zero_()


def _time_calls(fn, reps: int, warmup: int, flush: bool = False):
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    times = []
    for i in range(reps):
        if flush:
            flush_l2()
        else:
            torch.cuda._sleep(60000)      # keeps the GPU busy (~30 us) while the host enqueues, so that the event pair
                                          # brackets the kernel and not the host's launch latency
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn(i)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    return times


def layer_roofline(Mg, Ng, ab, wb, conv, R, S, C, in_rows, ms, popc_per_s, hbm_gbs):
    """Roofline of one contraction launch: the slower of its algorithmic bytes at the HBM peak (packed activations of
    the `in_rows` input rows or pixels and packed weights read once, fp32 outputs written once) and its popcount
    instructions at the measured popcount rate (the scarce pipe; qnn_popcounts_per_output per output element)."""
    kg = R * S * C
    nbytes = in_rows * C * ab / 8.0 + Ng * kg * wb / 8.0 + Mg * Ng * 4.0
    popc = qnn.popcounts_per_output(ab, wb, conv, R, S, C, Ng)
    t_alu = Mg * Ng * popc / popc_per_s * 1e3
    t_hbm = nbytes / (hbm_gbs * 1e9) * 1e3
    bound = "alu" if t_alu >= t_hbm else "hbm"
    binary = 2.0 * Mg * Ng * kg * ab * wb
    if bound == "alu":
        achieved, peak, unit = binary / (ms * 1e-3) / 1e12, binary / (t_alu * 1e-3) / 1e12, "binary TOPS"
    else:
        achieved, peak, unit = nbytes / (ms * 1e-3) / 1e9, hbm_gbs, "GB/s"
    return {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": max(t_alu, t_hbm) / ms,
            "roofline_ms": max(t_alu, t_hbm), "popc_per_word": popc / (ab * wb * (kg / 32.0)), "alg_bytes": nbytes}


def time_gemm(Mg, Ng, Kg, ab, wb, reps=5, warmup=3, sets=3, dev="cuda:0", seed=0):
    g = torch.Generator(device=dev).manual_seed(seed)
    w = torch.randn((Ng, Kg), device=dev, generator=g) * 0.02
    sw = float(w.abs().max()) / (2 ** wb - 1)
    packed = qnn.pack_weights(w, Ng, 1, Kg, qnn.W_NTC, wb, sw)
    planes, outs = [], []
    for _ in range(sets):
        a = torch.randn((Mg, Kg), device=dev, generator=g).abs_().clamp_(max=4.0)
        planes.append(qnn.encode_pack(a, ab, 4.0 / (2 ** ab - 1)))
        outs.append(torch.empty((Mg, Ng), dtype=torch.float32, device=dev))
        del a
    times = _time_calls(lambda i: qnn.bgemm(planes[i % sets], ab, packed, wb, Mg, Ng, Kg, 1e-3, out=outs[i % sets]),
                        reps, warmup)
    return _report("qnn_bgemm", Mg, Ng, Kg, ab, wb, times)


def time_conv(N, H, W, C, Cout, R, S, stride, pad, ab, wb, reps=5, warmup=3, sets=2, dev="cuda:0", seed=0):
    g = torch.Generator(device=dev).manual_seed(seed)
    w = torch.randn((Cout, R, S, C), device=dev, generator=g) * 0.02
    sw = float(w.abs().max()) / (2 ** wb - 1)
    packed = qnn.pack_weights(w, Cout, R * S, C, qnn.W_NTC, wb, sw)
    Ho, Wo = qnn.conv_out_dim(H, R, stride, pad), qnn.conv_out_dim(W, S, stride, pad)
    planes, outs = [], []
    for _ in range(sets):
        a = torch.randn((N * H * W, C), device=dev, generator=g).clamp_(min=0.0)
        planes.append(qnn.encode_pack(a, ab, 4.0 / (2 ** ab - 1)))
        outs.append(torch.empty((N, Ho, Wo, Cout), dtype=torch.float32, device=dev))
        del a
    times = _time_calls(lambda i: qnn.bconv2d(planes[i % sets], ab, packed, wb, N, H, W, C, Cout, R, S, stride, pad,
                                              1e-3, out=outs[i % sets]), reps, warmup)
    return _report("qnn_bconv2d", N * Ho * Wo, Cout, R * S * C, ab, wb, times)


def time_encode(rows, k, bits, reps=5, warmup=3, sets=3, relu=False, dev="cuda:0", seed=0):
    g = torch.Generator(device=dev).manual_seed(seed)
    xs = [torch.randn((rows, k), device=dev, generator=g) for _ in range(sets)]
    planes = [torch.empty((rows, bits, qnn.row_words(k)), dtype=torch.int32, device=dev) for _ in range(sets)]
    times = _time_calls(lambda i: qnn.encode_pack(xs[i % sets], bits, 0.37, qnn.RELU if relu else 0,
                                                  planes=planes[i % sets]), reps, warmup)
    ms = statistics.median(times)
    nbytes = rows * k * 4 + rows * bits * qnn.row_words(k) * 4
    return {"call": "qnn_encode_pack", "rows": rows, "k": k, "bits": bits, "ms_median": ms, "ms_min": min(times),
            "bytes": nbytes, "gbs": nbytes / (ms * 1e-3) / 1e9}


def time_stack(net: str, batch: int, reps=3, warmup=2, dev="cuda:0", seed=0, layers=None):
    """Every quantized convolution of a ResNet-18- or VGG-16-shaped stack, each on its own synthetic
    input of the right shape (post-ReLU half-normal), timed as qnn_encode_pack + qnn_bconv2d."""
    from . import workloads as wl
    if net == "resnet18":
        shapes = wl.resnet18_shapes(batch)
    elif net in ("resnet18_p1", "resnet18_p2"):
        shapes = wl.resnet18_mixed_shapes(int(net[-1]), batch)     # Table 4's mixed precisions
    else:
        shapes = wl.vgg16_shapes(batch)
    g = torch.Generator(device=dev).manual_seed(seed)
    rows = []
    for li, s in enumerate(shapes):
        if layers is not None and li not in layers:
            continue
        w = torch.randn((s.Cout, s.R, s.S, s.C), device=dev, generator=g) * (2.0 / (s.R * s.S * s.C)) ** 0.5
        packed = qnn.pack_weights(w, s.Cout, s.R * s.S, s.C, qnn.W_NTC, s.wb, float(w.abs().max()) / (2 ** s.wb - 1))
        a = torch.randn((s.N * s.H * s.W, s.C), device=dev, generator=g)
        planes = torch.empty((s.N * s.H * s.W, s.ab, qnn.row_words(s.C)), dtype=torch.int32, device=dev)
        out = torch.empty((s.N, s.Ho, s.Wo, s.Cout), dtype=torch.float32, device=dev)
        sa = 4.0 / (2 ** s.ab - 1)
        t_enc = _time_calls(lambda i: qnn.encode_pack(a, s.ab, sa, qnn.RELU, planes=planes), reps, warmup)
        t_conv = _time_calls(lambda i: qnn.bconv2d(planes, s.ab, packed, s.wb, s.N, s.H, s.W, s.C, s.Cout, s.R, s.S,
                                                   s.stride, s.pad, 1e-3, out=out), reps, warmup)
        # layer chaining: the same convolution writing the next layer's planes instead of fp32
        nxt = torch.empty((s.Mg, s.ab, qnn.row_words(s.Cout)), dtype=torch.int32, device=dev)
        fused_out = out if (s.R * s.S * s.C <= 32) else None      # single-word patches encode from the fp32 result
        t_fused = _time_calls(lambda i: qnn.bconv2d_encode(planes, s.ab, packed, s.wb, s.N, s.H, s.W, s.C, s.Cout, s.R,
                                                           s.S, s.stride, s.pad, 1e-3, s.ab, sa, qnn.RELU,
                                                           next_planes=nxt, out=fused_out), reps, warmup)
        del nxt
        enc_ms, conv_ms = statistics.median(t_enc), statistics.median(t_conv)
        macs = float(s.Mg) * s.Cout * s.Kg
        rows.append({"layer": s.name, "Mg": s.Mg, "Ng": s.Cout, "Kg": s.Kg, "ab": s.ab, "wb": s.wb,
                     "R": s.R, "S": s.S, "C": s.C, "stride": s.stride, "in_rows": s.N * s.H * s.W,
                     "encode_ms": enc_ms, "conv_ms": conv_ms, "conv_encode_ms": statistics.median(t_fused),
                     "conv_binary_tops": 2 * macs * s.ab * s.wb / (conv_ms * 1e-3) / 1e12,
                     "conv_equiv_int_gops": 2 * macs / (conv_ms * 1e-3) / 1e9,
                     "encode_gbs": (a.numel() * 4 + planes.numel() * 4) / (enc_ms * 1e-3) / 1e9,
                     "out_bytes": out.numel() * 4, "in_bytes_fp32": a.numel() * 4, "int_macs": macs})
        del a, planes, out, w, packed
    tot_ms = sum(r["encode_ms"] + r["conv_ms"] for r in rows)
    tot_macs = sum(r["int_macs"] for r in rows)
    bin_macs = sum(r["int_macs"] * r["ab"] * r["wb"] for r in rows)
    return {"call": f"stack:{net}", "batch": batch, "layers": rows, "total_ms": tot_ms,
            "binary_tops": 2 * bin_macs / (tot_ms * 1e-3) / 1e12, "equiv_int_gops": 2 * tot_macs / (tot_ms * 1e-3) / 1e9}


def time_mbit(n, bits, reps=5, warmup=3, dev="cuda:0", seed=0):
    """Trigonometric encoder forward and backward on n elements (streaming kernels; GB/s of their algorithmic bytes)."""
    g = torch.Generator(device=dev).manual_seed(seed)
    x = torch.rand(n, device=dev, generator=g) * 2 - 1
    c = torch.empty((bits, n), dtype=torch.float32, device=dev)
    gc = torch.randn((bits, n), device=dev, generator=g)
    gx = torch.empty(n, dtype=torch.float32, device=dev)
    tf = statistics.median(_time_calls(lambda i: qnn.mbit_encoder_forward(x, bits, 1.0, c=c), reps, warmup))
    tb = statistics.median(_time_calls(lambda i: qnn.mbit_encoder_backward(x, gc, bits, 1.0, gx=gx), reps, warmup))
    return {"call": "qnn_mbit_encoder", "n": n, "bits": bits, "forward_ms": tf, "backward_ms": tb,
            "forward_gbs": n * 4 * (1 + bits) / (tf * 1e-3) / 1e9, "backward_gbs": n * 4 * (2 + bits) / (tb * 1e-3) / 1e9}


def time_backward(m, n, k, ab, wb, reps=5, warmup=3, dev="cuda:0", seed=0):
    """Backward products of one FC layer (TF32 tensor-core contractions): whole calls, and the staging part alone."""
    g = torch.Generator(device=dev).manual_seed(seed)
    grad = torch.randn((m, n), device=dev, generator=g)
    x = (torch.rand((m, k), device=dev, generator=g) * 2 - 1)
    a_planes = qnn.encode_pack(x, ab, 1.0 / (2 ** ab - 1))
    w_planes = qnn.encode_pack(torch.randn((n, k), device=dev, generator=g).clamp_(-1, 1), wb, 1.0 / (2 ** wb - 1))
    alpha = 1.0 / ((2 ** ab - 1) * (2 ** wb - 1))
    out = torch.empty((m, k), dtype=torch.float32, device=dev)
    gw = torch.empty((n, k), dtype=torch.float32, device=dev)
    wsd = torch.empty(qnn.lib.qnn_bgemm_backward_data_workspace(m, n, k) + 256, dtype=torch.uint8, device=dev)
    wsw = torch.empty(qnn.lib.qnn_bgemm_backward_weights_workspace(m, n, k) + 256, dtype=torch.uint8, device=dev)
    med = lambda f: statistics.median(_time_calls(f, reps, warmup))
    td = med(lambda i: qnn.bgemm_backward_data(grad, w_planes, k, wb, alpha, out=out, workspace=wsd))
    te = med(lambda i: qnn.bgemm_backward_data(grad, w_planes, k, wb, alpha, x=x, ab=ab, r=1.0, out=out, workspace=wsd))
    tw = med(lambda i: qnn.bgemm_backward_weights(grad, a_planes, k, ab, alpha, gw=gw, workspace=wsw))
    tu = med(lambda i: qnn.unpack_codes_f32(w_planes, n, k, wb, transpose=True))
    status = qnn.tensor_path_status()
    fl = 2.0 * m * n * k
    return {"call": "qnn_bgemm_backward", "m": m, "n": n, "k": k, "ab": ab, "wb": wb, "status": status,
            "data_ms": td, "data_encoder_ms": te, "weights_ms": tw, "unpack_t_ms": tu,
            "data_tflops": fl / (td * 1e-3) / 1e12, "data_encoder_tflops": fl / (te * 1e-3) / 1e12,
            "weights_tflops": fl / (tw * 1e-3) / 1e12}


def time_backward_conv(N, H, W, C, Cout, R, S, stride, pad, ab, wb, reps=5, warmup=3, dev="cuda:0", seed=0):
    """Backward products of one convolution layer: whole calls (patch staging + TF32 tensor-core GEMM + gather)."""
    g = torch.Generator(device=dev).manual_seed(seed)
    Ho, Wo = qnn.conv_out_dim(H, R, stride, pad), qnn.conv_out_dim(W, S, stride, pad)
    grad = torch.randn((N, Ho, Wo, Cout), device=dev, generator=g)
    x = torch.rand((N * H * W, C), device=dev, generator=g) * 2 - 1
    a_planes = qnn.encode_pack(x, ab, 1.0 / (2 ** ab - 1))
    w = torch.randn((Cout, R, S, C), device=dev, generator=g).clamp_(-1, 1)
    packed = qnn.pack_weights(w, Cout, R * S, C, qnn.W_NTC, wb, 1.0 / (2 ** wb - 1))
    alpha = 1.0 / ((2 ** ab - 1) * (2 ** wb - 1))
    out = torch.empty((N, H, W, C), dtype=torch.float32, device=dev)
    gw = torch.empty((Cout, R, S, C), dtype=torch.float32, device=dev)
    wsd = torch.empty(qnn.lib.qnn_bconv2d_backward_data_workspace(N, H, W, C, Cout, R, S, stride, pad) + 256, dtype=torch.uint8, device=dev)
    wsw = torch.empty(qnn.lib.qnn_bconv2d_backward_weights_workspace(N, H, W, C, Cout, R, S, stride, pad) + 256, dtype=torch.uint8, device=dev)
    med = lambda f: statistics.median(_time_calls(f, reps, warmup))
    td = med(lambda i: qnn.bconv2d_backward_data(grad, packed, wb, H, W, C, R, S, stride, pad, alpha, out=out, workspace=wsd))
    tw = med(lambda i: qnn.bconv2d_backward_weights(grad, a_planes, ab, H, W, C, R, S, stride, pad, alpha, gw=gw, workspace=wsw))
    status = qnn.tensor_path_status()
    fl = 2.0 * N * Ho * Wo * Cout * R * S * C
    return {"call": "qnn_bconv2d_backward", "N": N, "H": H, "W": W, "C": C, "Cout": Cout, "R": R, "S": S, "stride": stride,
            "pad": pad, "ab": ab, "wb": wb, "status": status, "data_ms": td, "weights_ms": tw,
            "data_tflops": fl / (td * 1e-3) / 1e12, "weights_tflops": fl / (tw * 1e-3) / 1e12,
            "workspace_mb": [wsd.numel() / 1e6, wsw.numel() / 1e6]}


def _report(call, Mg, Ng, Kg, ab, wb, times):
    ms = statistics.median(times)
    macs = float(Mg) * Ng * Kg
    return {"call": call, "Mg": Mg, "Ng": Ng, "Kg": Kg, "ab": ab, "wb": wb, "ms_median": ms, "ms_min": min(times),
            "binary_tops": 2 * macs * ab * wb / (ms * 1e-3) / 1e12, "equiv_int_gops": 2 * macs / (ms * 1e-3) / 1e9,
            "bytes": Mg * Kg * ab / 8 + Ng * Kg * wb / 8 + Mg * Ng * 4}


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="case", required=True)
    g = sub.add_parser("gemm")
    for name, default in (("m", 4096), ("n", 4096), ("k", 4096), ("ab", 2), ("wb", 2)):
        g.add_argument(f"--{name}", type=int, default=default)
    c = sub.add_parser("conv")
    for name, default in (("N", 32), ("H", 14), ("W", 14), ("C", 256), ("Cout", 256), ("R", 3), ("S", 3),
                          ("stride", 1), ("pad", 1), ("ab", 2), ("wb", 2)):
        c.add_argument(f"--{name}", type=int, default=default)
    e = sub.add_parser("encode")
    for name, default in (("rows", 4096), ("k", 4096), ("bits", 2)):
        e.add_argument(f"--{name}", type=int, default=default)
    mb = sub.add_parser("mbit")
    mb.add_argument("--n", type=int, default=1 << 26)
    mb.add_argument("--bits", type=int, default=2)
    bw = sub.add_parser("backward")
    bw.add_argument("--m", type=int, default=4096)
    bw.add_argument("--n", type=int, default=4096)
    bw.add_argument("--k", type=int, default=4096)
    bw.add_argument("--ab", type=int, default=2)
    bw.add_argument("--wb", type=int, default=2)
    bc = sub.add_parser("backward_conv")
    for name, default in (("N", 32), ("H", 14), ("W", 14), ("C", 256), ("Cout", 256), ("R", 3), ("S", 3),
                          ("stride", 1), ("pad", 1), ("ab", 2), ("wb", 2)):
        bc.add_argument(f"--{name}", type=int, default=default)
    k = sub.add_parser("stack")
    k.add_argument("--net", choices=["resnet18", "resnet18_p1", "resnet18_p2", "vgg16"], default="resnet18")
    k.add_argument("--batch", type=int, default=0)
    k.add_argument("--layers", type=str, default="")
    k.add_argument("--table", action="store_true")
    for s in (g, c, e, k, mb, bw, bc):
        s.add_argument("--reps", type=int, default=5)
        s.add_argument("--warmup", type=int, default=3)
        s.add_argument("--sets", type=int, default=3)
    a = ap.parse_args()
    if a.case == "gemm":
        r = time_gemm(a.m, a.n, a.k, a.ab, a.wb, a.reps, a.warmup, a.sets)
    elif a.case == "conv":
        r = time_conv(a.N, a.H, a.W, a.C, a.Cout, a.R, a.S, a.stride, a.pad, a.ab, a.wb, a.reps, a.warmup, a.sets)
    elif a.case == "backward":
        r = time_backward(a.m, a.n, a.k, a.ab, a.wb, a.reps, a.warmup)
    elif a.case == "backward_conv":
        r = time_backward_conv(a.N, a.H, a.W, a.C, a.Cout, a.R, a.S, a.stride, a.pad, a.ab, a.wb, a.reps, a.warmup)
    elif a.case == "mbit":
        r = time_mbit(a.n, a.bits, a.reps, a.warmup)
    elif a.case == "stack":
        batch = a.batch or (64 if a.net == "vgg16" else 256)
        layers = [int(v) for v in a.layers.split(",")] if a.layers else None
        r = time_stack(a.net, batch, a.reps, a.warmup, layers=layers)
        if a.table:
            print(f"{'layer':28s} {'Mg':>8s} {'Ng':>4s} {'Kg':>5s} {'enc ms':>8s} {'conv ms':>8s} {'bTOPS':>7s} {'enc GB/s':>8s} {'conv+enc fused ms':>18s}")
            for L in r["layers"]:
                print(f"{L['layer']:28s} {L['Mg']:8d} {L['Ng']:4d} {L['Kg']:5d} {L['encode_ms']:8.3f} {L['conv_ms']:8.3f} "
                      f"{L['conv_binary_tops']:7.1f} {L['encode_gbs']:8.0f} {L['conv_encode_ms']:18.3f}")
            print(f"total {r['total_ms']:.3f} ms (encode + conv per layer), {r['binary_tops']:.1f} binary TOPS, "
                  f"{r['equiv_int_gops']:.0f} equiv int GOPS; chained plane-to-plane (fused encoder, no fp32 between "
                  f"layers): {sum(L['conv_encode_ms'] for L in r['layers']):.3f} ms")
            return
    else:
        r = time_encode(a.rows, a.k, a.bits, a.reps, a.warmup, a.sets)
    print(json.dumps(r))


if __name__ == "__main__":
    main()

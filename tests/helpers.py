"""Shared drivers for the parity tests: run one layer through the oracle and through libqnn."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2106_09886_b200 import workloads as wl


def scales_for(a, w, ab, wb):
    sa, sw = wl.per_tensor_scale(a, ab), wl.per_tensor_scale(w, wb)
    return sa, sw, np.float32(sa * sw)


# ---------------------------------------------------------------- oracle side

def oracle_fc_codes(a, w, k_major, ab, wb, sa, sw, relu=False):
    qa = oracle.quantize(a, ab, sa, relu)
    qw = oracle.quantize(w, wb, sw)
    if k_major:
        qw = np.ascontiguousarray(qw.T)
    return qa, qw


def oracle_fc(a, w, k_major, ab, wb, sa, sw, alpha, relu=False):
    qa, qw = oracle_fc_codes(a, w, k_major, ab, wb, sa, sw, relu)
    acc = oracle.fc(qa, qw)
    return qa, qw, acc, oracle.scale(acc, alpha)


def oracle_conv(a, w, ab, wb, sa, sw, alpha, stride, pad, relu=False):
    qa = oracle.quantize(a, ab, sa, relu)
    qw = oracle.quantize(w, wb, sw)
    acc = oracle.conv2d(qa, qw, stride, pad)
    return qa, qw, acc, oracle.scale(acc, alpha)


def oracle_weight_planes(qw_ntc, bits):
    """Codes [n_out, taps, c] -> (planes uint32 [n_out, bits, row_words], tapsum [n_out, taps]) in the
    packed-weights geometry (each tap starts on a word boundary), built from the oracle's canonical packer."""
    n_out, taps, c = qw_ntc.shape
    cw = (c + 31) // 32
    per_tap = oracle.pack_planes(qw_ntc.reshape(n_out * taps, c), bits)[:, :, :cw]     # [n*taps, bits, cw]
    per_tap = per_tap.reshape(n_out, taps, bits, cw).transpose(0, 2, 1, 3).reshape(n_out, bits, taps * cw)
    kw = (taps * cw + 3) // 4 * 4
    planes = np.zeros((n_out, bits, kw), dtype=np.uint32)
    planes[:, :, :taps * cw] = per_tap
    t = (qw_ntc.astype(np.int64) + (2 ** bits - 1)) // 2
    return planes, t.sum(axis=2).astype(np.int32)


# ---------------------------------------------------------------- GPU side

def gpu_fc(a, w, k_major, ab, wb, sa, sw, alpha, relu=False, want_planes=False):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    Mg, Kg = a.shape
    Ng = w.shape[1] if k_major else w.shape[0]
    a_d = torch.from_numpy(a).to(dev)
    w_d = torch.from_numpy(np.ascontiguousarray(w)).to(dev)
    planes = qnn.encode_pack(a_d, ab, sa, qnn.RELU if relu else 0)
    packed = qnn.pack_weights(w_d, Ng, 1, Kg, qnn.W_TCN if k_major else qnn.W_NTC, wb, sw)
    out, acc = qnn.bgemm(planes, ab, packed, wb, Mg, Ng, Kg, alpha, want_acc=True)
    torch.cuda.synchronize()
    res = {"out": out.cpu().numpy(), "acc": acc.cpu().numpy()}
    if want_planes:
        wp, ts = qnn.weights_views(packed, Ng, 1, Kg, wb)
        res["a_planes"] = planes.cpu().numpy().view(np.uint32)
        res["w_planes"] = wp.cpu().numpy().view(np.uint32)
        res["tapsum"] = ts.cpu().numpy()
    return res


def gpu_conv(a, w, ab, wb, sa, sw, alpha, stride, pad, relu=False, want_planes=False):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    N, H, W, C = a.shape
    Cout, R, S, _ = w.shape
    a_d = torch.from_numpy(a).to(dev)
    w_d = torch.from_numpy(w).to(dev)
    planes = qnn.encode_pack(a_d.view(N * H * W, C), ab, sa, qnn.RELU if relu else 0)
    packed = qnn.pack_weights(w_d, Cout, R * S, C, qnn.W_NTC, wb, sw)
    out, acc = qnn.bconv2d(planes, ab, packed, wb, N, H, W, C, Cout, R, S, stride, pad, alpha, want_acc=True)
    torch.cuda.synchronize()
    res = {"out": out.cpu().numpy(), "acc": acc.cpu().numpy()}
    if want_planes:
        wp, ts = qnn.weights_views(packed, Cout, R * S, C, wb)
        res["a_planes"] = planes.cpu().numpy().view(np.uint32)
        res["w_planes"] = wp.cpu().numpy().view(np.uint32)
        res["tapsum"] = ts.cpu().numpy()
    return res


def assert_fp32_close(got, want, rtol=1e-6):
    """fp32 outputs: within 1e-6 relative (they are single correctly-rounded products, so normally equal)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape
    err = np.abs(got - want)
    tol = rtol * np.abs(want)
    assert np.all(err <= tol), f"max rel err {np.max(err / np.maximum(np.abs(want), 1e-30))}"

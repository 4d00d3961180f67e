"""GPU parity of the fused layer chaining calls (qnn_bgemm_encode / qnn_bconv2d_encode): the next layer's bit
planes written by the contraction's epilogue must equal, bit for bit, the oracle's quantize + pack applied to
the oracle's fp32 result (ReLU fused), padding words included."""
import numpy as np
import pytest

import oracle
from helpers import assert_fp32_close, oracle_conv, oracle_fc, scales_for
from paper_2106_09886_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _env():
    import torch
    from paper_2106_09886_b200 import qnn
    return torch, qnn, torch.device("cuda:0")


@pytest.mark.parametrize("Mg,Ng,Kg,ab,wb,nb", [
    (1, 1, 40, 2, 2, 2), (70, 17, 300, 2, 2, 3), (64, 64, 512, 2, 2, 2), (130, 65, 129, 3, 3, 3), (200, 100, 700, 4, 4, 4),
    (33, 130, 96, 1, 1, 1), (257, 260, 1000, 2, 4, 8), (90, 128, 640, 5, 3, 2), (45, 200, 333, 8, 8, 5)])
def test_bgemm_encode(Mg, Ng, Kg, ab, wb, nb):
    torch, qnn, dev = _env()
    rng = np.random.default_rng(Mg + 7 * Ng + Kg)
    a = rng.standard_normal((Mg, Kg)).astype(np.float32)
    w = rng.standard_normal((Ng, Kg)).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_fc(a, w, False, ab, wb, sa, sw, alpha)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev), ab, sa)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Ng, 1, Kg, qnn.W_NTC, wb, sw)
    for relu in (True, False):
        act = np.maximum(out, 0) if relu else out
        ns = wl.per_tensor_scale(act, nb)
        want = oracle.pack_planes(oracle.quantize(out, nb, ns, relu), nb)
        for with_out in (False, True):
            nxt = torch.full((Mg, nb, qnn.row_words(Ng)), -1, dtype=torch.int32, device=dev)
            out_d = torch.full((Mg, Ng), 7.0, dtype=torch.float32, device=dev) if with_out else None
            qnn.bgemm_encode(planes, ab, packed, wb, Mg, Ng, Kg, alpha, nb, ns, qnn.RELU if relu else 0,
                             next_planes=nxt, out=out_d)
            torch.cuda.synchronize()
            assert np.array_equal(nxt.cpu().numpy().view(np.uint32), want)
            if with_out:
                assert_fp32_close(out_d.cpu().numpy(), out)


@pytest.mark.parametrize("N,H,W,C,Cout,R,S,stride,pad,ab,wb,nb", [
    (2, 9, 10, 64, 70, 3, 3, 1, 1, 3, 3, 3), (1, 14, 14, 128, 33, 3, 3, 2, 1, 2, 2, 2), (2, 8, 8, 256, 64, 1, 1, 2, 0, 3, 3, 3),
    (1, 17, 13, 100, 129, 3, 3, 1, 1, 4, 4, 4), (2, 12, 12, 3, 64, 3, 3, 1, 1, 4, 4, 4), (1, 7, 7, 512, 200, 3, 3, 1, 1, 2, 4, 1)])
def test_bconv2d_encode(N, H, W, C, Cout, R, S, stride, pad, ab, wb, nb):
    torch, qnn, dev = _env()
    rng = np.random.default_rng(N * 100 + H + C + Cout)
    a = rng.standard_normal((N, H, W, C)).astype(np.float32)
    w = (0.05 * rng.standard_normal((Cout, R, S, C))).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_conv(a, w, ab, wb, sa, sw, alpha, stride, pad, relu=True)
    ns = wl.per_tensor_scale(np.maximum(out, 0), nb)
    want = oracle.pack_planes(oracle.quantize(out.reshape(-1, Cout), nb, ns, True), nb)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev).view(-1, C), ab, sa, qnn.RELU)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Cout, R * S, C, qnn.W_NTC, wb, sw)
    Mg = out.shape[0] * out.shape[1] * out.shape[2]
    nxt = torch.full((Mg, nb, qnn.row_words(Cout)), -1, dtype=torch.int32, device=dev)
    out_d = torch.empty(out.shape, dtype=torch.float32, device=dev)
    qnn.bconv2d_encode(planes, ab, packed, wb, N, H, W, C, Cout, R, S, stride, pad, alpha, nb, ns, qnn.RELU,
                       next_planes=nxt, out=out_d)
    torch.cuda.synchronize()
    assert np.array_equal(nxt.cpu().numpy().view(np.uint32), want)
    assert_fp32_close(out_d.cpu().numpy(), out)


def test_resnet_stage_chained_without_fp32():
    """Four 3x3 convolutions of a ResNet-18-shaped stage, 3x3 bits, batch 2, chained plane to plane: no fp32
    tensor is written between the layers.  Scales are fixed beforehand from the oracle's own forward pass."""
    torch, qnn, dev = _env()
    shapes = [s for s in wl.resnet18_shapes(batch=2) if not s.branch][:5]
    x = wl.layer_input(0, 4, 200, shapes[0])
    # calibration + expectation on the oracle side
    ws, scales, alphas, want_planes = [], [], [], []
    cur = x
    for li, s in enumerate(shapes):
        w = wl.he_weights(0, 4, 300 + li, s)
        sa = wl.per_tensor_scale(np.maximum(cur, 0), s.ab)
        sw = wl.per_tensor_scale(w, s.wb)
        qa = oracle.quantize(cur, s.ab, sa, True)
        want_planes.append(oracle.pack_planes(qa.reshape(-1, s.C), s.ab))
        alpha = np.float32(sa * sw)
        cur = oracle.scale(oracle.conv2d(qa, oracle.quantize(w, s.wb, sw), s.stride, s.pad), alpha)
        ws.append((w, sw)); scales.append(sa); alphas.append(alpha)
    final_out = cur
    # library side: encode once, then plane -> plane
    planes = qnn.encode_pack(torch.from_numpy(x).to(dev).view(-1, shapes[0].C), shapes[0].ab, scales[0], qnn.RELU)
    for li, s in enumerate(shapes):
        assert np.array_equal(planes.cpu().numpy().view(np.uint32), want_planes[li]), s.name
        w, sw = ws[li]
        packed = qnn.pack_weights(torch.from_numpy(w).to(dev), s.Cout, s.R * s.S, s.C, qnn.W_NTC, s.wb, sw)
        if li + 1 < len(shapes):
            planes = qnn.bconv2d_encode(planes, s.ab, packed, s.wb, s.N, s.H, s.W, s.C, s.Cout, s.R, s.S, s.stride, s.pad,
                                        alphas[li], shapes[li + 1].ab, scales[li + 1], qnn.RELU)
        else:
            out = qnn.bconv2d(planes, s.ab, packed, s.wb, s.N, s.H, s.W, s.C, s.Cout, s.R, s.S, s.stride, s.pad, alphas[li])
            torch.cuda.synchronize()
            assert_fp32_close(out.cpu().numpy(), final_out)


def test_fused_argument_errors():
    torch, qnn, dev = _env()
    import ctypes
    x = torch.zeros((8, 64), dtype=torch.float32, device=dev)
    planes = qnn.encode_pack(x, 2, 1.0)
    packed = qnn.pack_weights(torch.ones((8, 64), dtype=torch.float32, device=dev), 8, 1, 64, qnn.W_NTC, 2, 1.0)
    nxt = torch.zeros((8, 2, 4), dtype=torch.int32, device=dev)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    f = qnn.lib.qnn_bgemm_encode
    assert f(p(planes), 2, p(packed), 2, 8, 8, 64, 1.0, None, None, 2, 1.0, 0, None, None, 8, None) == qnn.E_ARG
    assert f(p(planes), 2, p(packed), 2, 8, 8, 64, 1.0, None, None, 9, 1.0, 0, p(nxt), None, 8, None) == qnn.E_ARG
    assert f(p(planes), 2, p(packed), 2, 8, 8, 64, 1.0, None, None, 2, 0.0, 0, p(nxt), None, 8, None) == qnn.E_SCALE
    assert f(p(planes), 2, p(packed), 2, 8, 8, 64, 1.0, None, None, 2, 1.0, 4, p(nxt), None, 8, None) == qnn.E_ARG
    g = torch.ones(8, dtype=torch.float32, device=dev)
    assert f(p(planes), 2, p(packed), 2, 8, 8, 64, 1.0, None, p(g), 2, 1.0, 0, p(nxt), None, 8, None) == qnn.E_ARG   # beta without gamma
    assert f(p(planes), 2, p(packed), 2, 8, 8, 64, 1.0, p(g), None, 2, 1.0, 0, None, None, 8, None) == qnn.E_ARG     # affine only needs out
    # single-word patches encode from the fp32 result and therefore need `out`
    a3 = qnn.encode_pack(torch.zeros((16, 3), dtype=torch.float32, device=dev), 2, 1.0)
    w3 = qnn.pack_weights(torch.ones((4, 9, 3), dtype=torch.float32, device=dev), 4, 9, 3, qnn.W_NTC, 2, 1.0)
    assert qnn.lib.qnn_bconv2d_encode(p(a3), 2, p(w3), 2, 1, 4, 4, 3, 4, 3, 3, 1, 1, 1.0, None, None, 2, 1.0, 0, p(nxt), None, None) == qnn.E_ARG


@pytest.mark.parametrize("with_beta", [True, False])
def test_bgemm_affine_then_encode(with_beta):
    """Folded batch-norm: alpha = 1, y = fma(acc, gamma[n], beta[n]); fp32 result and next planes both checked."""
    torch, qnn, dev = _env()
    rng = np.random.default_rng(5)
    Mg, Ng, Kg, ab, wb, nb = 150, 100, 500, 3, 2, 3
    a = rng.standard_normal((Mg, Kg)).astype(np.float32)
    w = rng.standard_normal((Ng, Kg)).astype(np.float32)
    sa, sw, _ = scales_for(a, w, ab, wb)
    _, _, acc, _ = oracle_fc(a, w, False, ab, wb, sa, sw, np.float32(1))
    gamma = (rng.standard_normal(Ng) * 1e-3).astype(np.float32)
    beta = rng.standard_normal(Ng).astype(np.float32) if with_beta else None
    y = oracle.affine(oracle.scale(acc, np.float32(1)), gamma, beta)
    ns = wl.per_tensor_scale(np.maximum(y, 0), nb)
    want = oracle.pack_planes(oracle.quantize(y, nb, ns, True), nb)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev), ab, sa)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Ng, 1, Kg, qnn.W_NTC, wb, sw)
    g_d = torch.from_numpy(gamma).to(dev)
    b_d = torch.from_numpy(beta).to(dev) if with_beta else None
    out_d = torch.empty((Mg, Ng), dtype=torch.float32, device=dev)
    nxt = qnn.bgemm_encode(planes, ab, packed, wb, Mg, Ng, Kg, 1.0, nb, ns, qnn.RELU, out=out_d, ch_gamma=g_d, ch_beta=b_d)
    torch.cuda.synchronize()
    assert np.array_equal(out_d.cpu().numpy(), y)
    assert np.array_equal(nxt.cpu().numpy().view(np.uint32), want)
    # affine only (no encoder)
    out2 = torch.empty((Mg, Ng), dtype=torch.float32, device=dev)
    qnn.bgemm_encode(planes, ab, packed, wb, Mg, Ng, Kg, 1.0, 0, 0.0, 0, out=out2, ch_gamma=g_d, ch_beta=b_d, encode=False)
    torch.cuda.synchronize()
    assert np.array_equal(out2.cpu().numpy(), y)


@pytest.mark.parametrize("C,Cout", [(64, 70), (3, 64)])
def test_bconv2d_affine(C, Cout):
    torch, qnn, dev = _env()
    rng = np.random.default_rng(C)
    a = rng.standard_normal((2, 10, 9, C)).astype(np.float32)
    w = (0.05 * rng.standard_normal((Cout, 3, 3, C))).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, 2, 2)
    _, _, acc, out = oracle_conv(a, w, 2, 2, sa, sw, alpha, 1, 1)
    gamma = rng.standard_normal(Cout).astype(np.float32)
    beta = rng.standard_normal(Cout).astype(np.float32)
    y = oracle.affine(out, gamma, beta)
    ns = wl.per_tensor_scale(np.maximum(y, 0), 2)
    want = oracle.pack_planes(oracle.quantize(y.reshape(-1, Cout), 2, ns, True), 2)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev).view(-1, C), 2, sa)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Cout, 9, C, qnn.W_NTC, 2, sw)
    out_d = torch.empty(out.shape, dtype=torch.float32, device=dev)
    nxt = qnn.bconv2d_encode(planes, 2, packed, 2, 2, 10, 9, C, Cout, 3, 3, 1, 1, alpha, 2, ns, qnn.RELU, out=out_d,
                             ch_gamma=torch.from_numpy(gamma).to(dev), ch_beta=torch.from_numpy(beta).to(dev))
    torch.cuda.synchronize()
    assert np.array_equal(out_d.cpu().numpy(), y)
    assert np.array_equal(nxt.cpu().numpy().view(np.uint32), want)

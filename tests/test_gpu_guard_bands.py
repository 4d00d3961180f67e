"""Out-of-bounds writes would be silent on a GPU, so every output of the library is placed between guard bands
(sentinel bytes before and after) and the bands must come back untouched, over ragged shapes that exercise
partial tiles, padded leading dimensions, reduction tails and every kernel family."""
import ctypes

import numpy as np
import pytest

pytestmark = pytest.mark.gpu
GUARD = 4096          # bytes on each side (multiple of 16 keeps the payload aligned)
SENT = 0xA5


class Guarded:
    """A device byte buffer [guard | payload | guard]; `ptr` points at the payload."""

    def __init__(self, torch, dev, nbytes):
        self.torch = torch
        self.nbytes = int(nbytes)
        pad = (-self.nbytes) % 16
        self.buf = torch.full((GUARD + self.nbytes + pad + GUARD,), SENT, dtype=torch.uint8, device=dev)
        self.ptr = ctypes.c_void_p(self.buf.data_ptr() + GUARD)

    def check(self, what):
        self.torch.cuda.synchronize()
        b = self.buf
        assert bool((b[:GUARD] == SENT).all()), f"{what}: wrote before the buffer"
        assert bool((b[GUARD + self.nbytes:] == SENT).all()), f"{what}: wrote past the buffer"

    def payload(self, dtype):
        return self.buf[GUARD:GUARD + self.nbytes].view(dtype)


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2106_09886_b200 import qnn
    return torch, qnn, torch.device("cuda:0")


@pytest.mark.parametrize("rows,k,bits", [(1, 1, 1), (7, 3, 4), (33, 64, 2), (5, 65, 8), (100, 129, 3), (257, 1000, 2), (4097, 40, 4)])
def test_encode_pack_stays_inside(env, rows, k, bits):
    torch, qnn, dev = env
    x = torch.randn((rows, k), device=dev)
    planes = Guarded(torch, dev, qnn.planes_bytes(rows, k, bits))
    rowsum = Guarded(torch, dev, rows * 4)
    rc = qnn.lib.qnn_encode_pack(ctypes.c_void_p(x.data_ptr()), rows, k, k, bits, 0.3, 1, planes.ptr, rowsum.ptr, None)
    assert rc == 0
    planes.check("planes"); rowsum.check("rowsum")
    assert not bool((planes.payload(torch.uint8) == SENT).all())


@pytest.mark.parametrize("n_out,taps,c,bits", [(1, 1, 1, 1), (5, 9, 3, 4), (64, 9, 64, 3), (33, 25, 40, 2), (130, 1, 777, 8)])
def test_pack_weights_stays_inside(env, n_out, taps, c, bits):
    torch, qnn, dev = env
    w = torch.randn((n_out, taps, c), device=dev)
    packed = Guarded(torch, dev, qnn.weights_bytes(n_out, taps, c, bits))
    assert qnn.lib.qnn_pack_weights(ctypes.c_void_p(w.data_ptr()), n_out, taps, c, 0, bits, 0.2, packed.ptr, None) == 0
    packed.check("packed weights")


@pytest.mark.parametrize("Mg,Ng,Kg,ab,wb", [(1, 1, 1, 1, 1), (63, 65, 100, 2, 2), (65, 63, 129, 3, 3), (130, 1, 1000, 4, 4),
                                            (17, 200, 520, 8, 8), (300, 129, 96, 5, 2), (31, 64, 4097, 2, 7)])
def test_bgemm_stays_inside(env, Mg, Ng, Kg, ab, wb):
    torch, qnn, dev = env
    planes = qnn.encode_pack(torch.randn((Mg, Kg), device=dev), ab, 0.3)
    packed = qnn.pack_weights(torch.randn((Ng, Kg), device=dev), Ng, 1, Kg, qnn.W_NTC, wb, 0.3)
    out = Guarded(torch, dev, Mg * Ng * 4)
    acc = Guarded(torch, dev, Mg * Ng * 4)
    nxt = Guarded(torch, dev, qnn.planes_bytes(Mg, Ng, 3))
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    assert qnn.lib.qnn_bgemm(p(planes), ab, p(packed), wb, Mg, Ng, Kg, 0.01, out.ptr, Ng, acc.ptr, None) == 0
    out.check("out"); acc.check("acc")
    out2 = Guarded(torch, dev, Mg * Ng * 4)
    assert qnn.lib.qnn_bgemm_encode(p(planes), ab, p(packed), wb, Mg, Ng, Kg, 0.01, None, None, 3, 0.5, 1, nxt.ptr, out2.ptr,
                                    Ng, None) == 0
    nxt.check("next planes"); out2.check("out (chained call)")
    assert bool((nxt.payload(torch.uint8) != SENT).any()) or Mg * Ng < 8


@pytest.mark.parametrize("N,H,W,C,Cout,R,S,stride,pad,dil,tr,op,ab,wb", [
    (1, 1, 1, 1, 1, 1, 1, 1, 0, 1, 0, 0, 1, 1), (2, 7, 9, 3, 65, 3, 3, 1, 1, 1, 0, 0, 4, 4), (1, 13, 11, 64, 33, 3, 3, 2, 1, 1, 0, 0, 3, 3),
    (2, 6, 6, 100, 130, 5, 3, 1, 2, 1, 0, 0, 2, 2), (1, 9, 9, 40, 17, 3, 3, 1, 2, 2, 0, 0, 2, 3), (2, 5, 4, 70, 66, 3, 3, 2, 1, 1, 1, 1, 2, 2),
    (1, 8, 8, 256, 31, 1, 1, 2, 0, 1, 0, 0, 8, 2)])
def test_bconv2d_stays_inside(env, N, H, W, C, Cout, R, S, stride, pad, dil, tr, op, ab, wb):
    torch, qnn, dev = env
    planes = qnn.encode_pack(torch.randn((N * H * W, C), device=dev), ab, 0.3)
    packed = qnn.pack_weights(torch.randn((Cout, R * S, C), device=dev), Cout, R * S, C, qnn.W_NTC, wb, 0.3)
    Ho = qnn.conv_general_out_dim(H, R, stride, pad, dil, bool(tr), op)
    Wo = qnn.conv_general_out_dim(W, S, stride, pad, dil, bool(tr), op)
    n = N * Ho * Wo * Cout
    out, acc = Guarded(torch, dev, n * 4), Guarded(torch, dev, n * 4)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    assert qnn.lib.qnn_bconv2d_general(p(planes), ab, p(packed), wb, N, H, W, C, Cout, R, S, stride, pad, dil, tr, op, 0.01,
                                       out.ptr, acc.ptr, None) == 0
    out.check("out"); acc.check("acc")
    if dil == 1 and not tr:
        nxt = Guarded(torch, dev, qnn.planes_bytes(N * Ho * Wo, Cout, 2))
        out2 = Guarded(torch, dev, n * 4)
        assert qnn.lib.qnn_bconv2d_encode(p(planes), ab, p(packed), wb, N, H, W, C, Cout, R, S, stride, pad, 0.01, None, None,
                                          2, 0.5, 1, nxt.ptr, out2.ptr, None) == 0
        nxt.check("next planes"); out2.check("out (chained call)")

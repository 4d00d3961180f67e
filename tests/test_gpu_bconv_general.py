"""GPU parity: dilated and transposed convolution (qnn_bconv2d_general) against the CPU oracle."""
import numpy as np
import pytest

import oracle
from helpers import assert_fp32_close, scales_for

pytestmark = pytest.mark.gpu

CASES = [
    # N, H, W, C, Cout, R, S, stride, pad, dil, transposed, out_pad, ab, wb
    (2, 9, 8, 64, 40, 3, 3, 1, 2, 2, False, 0, 2, 2), (1, 15, 15, 128, 70, 3, 3, 1, 4, 4, False, 0, 3, 3),
    (1, 11, 11, 40, 6, 3, 3, 2, 1, 3, False, 0, 4, 2), (2, 7, 7, 256, 64, 3, 3, 1, 1, 1, False, 0, 2, 2),
    (2, 5, 6, 64, 33, 3, 3, 2, 1, 1, True, 1, 2, 2), (1, 4, 4, 70, 65, 4, 4, 2, 1, 1, True, 0, 3, 3),
    (1, 6, 5, 32, 4, 3, 2, 3, 0, 1, True, 2, 2, 4), (1, 5, 5, 200, 130, 3, 3, 2, 2, 2, True, 0, 4, 4),
    (2, 7, 7, 512, 64, 2, 2, 2, 0, 1, True, 0, 2, 2), (2, 3, 3, 6, 2, 1, 1, 2, 0, 1, True, 1, 8, 8),
    (1, 9, 9, 3, 16, 3, 3, 1, 2, 2, False, 0, 2, 2)]


@pytest.mark.parametrize("N,H,W,C,Cout,R,S,stride,pad,dil,transposed,out_pad,ab,wb", CASES)
def test_bconv2d_general(N, H, W, C, Cout, R, S, stride, pad, dil, transposed, out_pad, ab, wb):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(H * 100 + C + Cout + stride)
    a = rng.standard_normal((N, H, W, C)).astype(np.float32)
    w = (0.05 * rng.standard_normal((Cout, R, S, C))).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    qa, qw = oracle.quantize(a, ab, sa), oracle.quantize(w, wb, sw)
    acc = oracle.conv2d_general(qa, qw, stride, pad, dil, transposed, out_pad)
    out = oracle.scale(acc, alpha)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev).view(-1, C), ab, sa)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Cout, R * S, C, qnn.W_NTC, wb, sw)
    out_d, acc_d = qnn.bconv2d_general(planes, ab, packed, wb, N, H, W, C, Cout, R, S, stride, pad, dil, transposed, out_pad,
                                       alpha, want_acc=True)
    torch.cuda.synchronize()
    assert acc_d.shape == acc.shape
    assert np.array_equal(acc_d.cpu().numpy(), acc)
    assert_fp32_close(out_d.cpu().numpy(), out)


def test_general_reduces_to_plain_conv_and_rejects_bad_arguments():
    import ctypes
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(1)
    a = rng.standard_normal((1, 8, 8, 64)).astype(np.float32)
    w = rng.standard_normal((16, 3, 3, 64)).astype(np.float32)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev).view(-1, 64), 2, 0.5)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), 16, 9, 64, qnn.W_NTC, 2, 0.5)
    o1 = qnn.bconv2d(planes, 2, packed, 2, 1, 8, 8, 64, 16, 3, 3, 2, 1, 0.25)
    o2 = qnn.bconv2d_general(planes, 2, packed, 2, 1, 8, 8, 64, 16, 3, 3, 2, 1, 1, False, 0, 0.25)
    torch.cuda.synchronize()
    assert torch.equal(o1, o2)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    f = qnn.lib.qnn_bconv2d_general
    assert f(p(planes), 2, p(packed), 2, 1, 8, 8, 64, 16, 3, 3, 2, 1, 0, 0, 0, 1.0, p(o1), None, None) == qnn.E_ARG   # dilation 0
    assert f(p(planes), 2, p(packed), 2, 1, 8, 8, 64, 16, 3, 3, 2, 1, 1, 0, 1, 1.0, p(o1), None, None) == qnn.E_ARG   # out_pad on a forward conv
    assert f(p(planes), 2, p(packed), 2, 1, 8, 8, 64, 16, 3, 3, 2, 1, 1, 1, 2, 1.0, p(o1), None, None) == qnn.E_ARG   # out_pad >= stride and dilation
    assert f(p(planes), 2, p(packed), 2, 1, 8, 8, 64, 16, 3, 3, 1, 0, 9, 0, 0, 1.0, p(o1), None, None) == qnn.E_ARG   # dilated kernel larger than the image

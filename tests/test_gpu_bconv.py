"""GPU parity: qnn_bconv2d (implicit im2col, zero padding of the encoded tensor) against the CPU oracle."""
import numpy as np
import pytest

import oracle
from helpers import assert_fp32_close, gpu_conv, oracle_conv, oracle_weight_planes, scales_for
from paper_2106_09886_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run_conv(a, w, ab, wb, stride, pad, relu=False):
    sa, sw, alpha = scales_for(a, w, ab, wb)
    qa, qw, acc, out = oracle_conv(a, w, ab, wb, sa, sw, alpha, stride, pad, relu)
    got = gpu_conv(a, w, ab, wb, sa, sw, alpha, stride, pad, relu, want_planes=True)
    N, H, W, C = a.shape
    Cout, R, S, _ = w.shape
    assert np.array_equal(got["a_planes"], oracle.pack_planes(qa.reshape(-1, C), ab))
    wp, ts = oracle_weight_planes(qw.reshape(Cout, R * S, C), wb)
    assert np.array_equal(got["w_planes"], wp) and np.array_equal(got["tapsum"], ts)
    assert np.array_equal(got["acc"], acc)
    assert_fp32_close(got["out"], out)


@pytest.mark.parametrize("N,H,W,C,Cout,R,S,stride,pad", [
    (2, 5, 6, 7, 4, 3, 3, 1, 1), (1, 7, 7, 3, 5, 3, 3, 2, 1), (2, 6, 6, 9, 3, 1, 1, 2, 0),
    (1, 4, 5, 33, 2, 3, 3, 1, 0), (1, 9, 8, 4, 3, 5, 3, 2, 2), (2, 3, 3, 8, 8, 3, 3, 1, 1),
    (3, 14, 14, 64, 70, 3, 3, 1, 1), (2, 14, 14, 128, 33, 3, 3, 2, 1), (2, 8, 8, 256, 64, 1, 1, 2, 0),
    (1, 17, 13, 100, 65, 3, 3, 1, 1), (1, 30, 30, 3, 64, 3, 3, 1, 1), (2, 7, 7, 512, 130, 3, 3, 1, 1),
    (1, 1, 1, 40, 3, 3, 3, 1, 1), (1, 12, 12, 160, 16, 7, 7, 2, 3)])
def test_bconv2d_shapes(N, H, W, C, Cout, R, S, stride, pad):
    rng = np.random.default_rng(N * 1000 + H * 100 + C + Cout)
    a = rng.standard_normal((N, H, W, C)).astype(np.float32)
    w = (0.02 * rng.standard_normal((Cout, R, S, C))).astype(np.float32)
    run_conv(a, w, 2, 2, stride, pad)
    run_conv(a, w, 3, 4, stride, pad, relu=True)


@pytest.mark.parametrize("ab,wb", [(1, 1), (2, 4), (4, 2), (3, 3), (4, 4), (8, 8), (5, 2)])
def test_bconv2d_bit_widths(ab, wb):
    rng = np.random.default_rng(ab * 10 + wb)
    a = np.maximum(rng.standard_normal((2, 9, 10, 96)), 0).astype(np.float32)
    w = (0.02 * rng.standard_normal((40, 3, 3, 96))).astype(np.float32)
    run_conv(a, w, ab, wb, 1, 1)


def test_bconv2d_border_counts_valid_taps_only():
    """All codes +max: every output equals C*A*B times the number of taps inside the image."""
    a = np.full((1, 6, 6, 40), 1e6, np.float32)
    w = np.full((5, 3, 3, 40), 1e6, np.float32)
    got = gpu_conv(a, w, 2, 2, np.float32(1), np.float32(1), np.float32(1), 1, 1)
    acc = got["acc"][0, :, :, 0]
    assert acc[0, 0] == 40 * 9 * 4 and acc[0, 3] == 40 * 9 * 6 and acc[3, 3] == 40 * 9 * 9 and acc[5, 5] == 40 * 9 * 4


def test_config2_conv_layer_full():
    c = wl.conv_config2(0)
    s = c.shape
    run_conv(c.a, c.w, s.ab, s.wb, s.stride, s.pad)

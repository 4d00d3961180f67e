"""GPU parity on randomly drawn shapes and bit widths (seeded): FC and convolution, including reductions that
end in 1..7-word tails, tiles with ragged rows/columns, strides, paddings, rectangular kernels."""
import numpy as np
import pytest

from helpers import assert_fp32_close, gpu_conv, gpu_fc, oracle_conv, oracle_fc, scales_for

pytestmark = pytest.mark.gpu


def _bits(rng):
    return int(rng.integers(1, 5)) if rng.random() < 0.8 else int(rng.integers(5, 9))


@pytest.mark.parametrize("seed", range(24))
def test_random_fc(seed):
    rng = np.random.default_rng(1000 + seed)
    Mg, Ng = int(rng.integers(1, 400)), int(rng.integers(1, 300))
    Kg = int(rng.choice([rng.integers(1, 64), rng.integers(64, 700), 32 * rng.integers(1, 40), rng.integers(700, 3000)]))
    ab, wb = _bits(rng), _bits(rng)
    a = rng.standard_normal((Mg, Kg)).astype(np.float32)
    w = rng.standard_normal((Ng, Kg)).astype(np.float32)
    relu = bool(rng.integers(0, 2))
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_fc(a, w, False, ab, wb, sa, sw, alpha, relu)
    got = gpu_fc(a, w, False, ab, wb, sa, sw, alpha, relu)
    assert np.array_equal(got["acc"], acc), (Mg, Ng, Kg, ab, wb)
    assert_fp32_close(got["out"], out)


@pytest.mark.parametrize("seed", range(32))
def test_random_conv(seed):
    rng = np.random.default_rng(2000 + seed)
    N = int(rng.integers(1, 4))
    H, W = int(rng.integers(1, 20)), int(rng.integers(1, 20))
    C = int(rng.choice([rng.integers(1, 8), rng.integers(8, 70), 32 * rng.integers(1, 9), rng.integers(70, 300)]))
    Cout = int(rng.integers(1, 150))
    R, S = int(rng.choice([1, 2, 3, 5])), int(rng.choice([1, 2, 3, 5]))
    stride = int(rng.integers(1, 4))
    pad = int(rng.integers(0, 3))
    if H + 2 * pad < R or W + 2 * pad < S:
        H, W = H + R, W + S
    ab, wb = _bits(rng), _bits(rng)
    a = rng.standard_normal((N, H, W, C)).astype(np.float32)
    w = rng.standard_normal((Cout, R, S, C)).astype(np.float32)
    relu = bool(rng.integers(0, 2))
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_conv(a, w, ab, wb, sa, sw, alpha, stride, pad, relu)
    got = gpu_conv(a, w, ab, wb, sa, sw, alpha, stride, pad, relu)
    assert np.array_equal(got["acc"], acc), (N, H, W, C, Cout, R, S, stride, pad, ab, wb)
    assert_fp32_close(got["out"], out)

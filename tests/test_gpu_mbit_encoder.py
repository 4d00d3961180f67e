"""GPU parity of the trigonometric M-bit encoder (Eq. 10) and its derivative (Eq. 12) against the CPU oracle.
Forward: exact (the sign is a decision taken in binary32 on both sides).  Backward: binary32 arithmetic against the
oracle's binary64.  The kernel rounds y = k_m*xn to binary32 before the cosine, an absolute error of at most
|y| * 2^-24 <= k_m * 2^-24 in y, hence pi * k_m * 2^-24 in cos(pi*y); cospif, the two products and the accumulation add
a few units of 2^-24 relative to each term.  So
    |got - want| <= sum_m |gc_m| * k_m * pi * (pi * k_m + 8) * 2^-24 / r."""
import math

import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bits", range(1, 9))
def test_forward_exact(bits):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(bits)
    A = 2 ** bits - 1
    x = rng.uniform(-1.2, 1.2, size=100003).astype(np.float32)
    # zero crossings and their neighbours, non-finite values
    cross = (np.arange(-A - 1, A + 2, dtype=np.float64) * 2.0 / A).astype(np.float32)
    special = np.concatenate([cross, np.nextafter(cross, np.float32(np.inf)), np.nextafter(cross, np.float32(-np.inf)),
                              np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 2.0, -2.0, 4.0], dtype=np.float32)])
    x[:special.size] = special
    for r in (1.0, 3.0, 0.37):
        want = oracle.mbit_encoder_forward(x, bits, r)
        got = qnn.mbit_encoder_forward(torch.from_numpy(x).to(dev), bits, r).cpu().numpy()
        assert np.array_equal(got, want), (bits, r)
    # away from crossings the outputs are the planes of the table encoder
    xi = x[np.isfinite(x) & (np.abs(x) <= 1)]
    xi = xi[np.abs(xi * A / 2 - np.round(xi * A / 2)) > 1e-3]
    c = qnn.mbit_encoder_forward(torch.from_numpy(xi).to(dev), bits, 1.0).cpu().numpy()
    planes = qnn.encode_pack(torch.from_numpy(xi).to(dev).view(1, -1), bits, 1.0 / A).cpu().numpy().view(np.uint32)
    k = np.arange(xi.size)
    for m in range(bits):
        b = (planes[0, m][k // 32] >> (k % 32).astype(np.uint32)) & 1
        assert np.array_equal(c[m], np.where(b == 1, 1.0, -1.0).astype(np.float32))


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 6, 8])
def test_backward_within_tolerance(bits):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(10 + bits)
    n = 70001
    x = rng.uniform(-1.3, 1.3, size=n).astype(np.float32)
    x[:6] = np.array([-1.0, 1.0, 0.0, 1.0000001, -1.0000001, 5.0], dtype=np.float32)
    gc = rng.standard_normal((bits, n)).astype(np.float32)
    A = 2 ** bits - 1
    for r in (1.0, 2.5):
        xr = (x * np.float32(r)).astype(np.float32)
        want = oracle.mbit_encoder_backward(xr, gc, bits, r)
        got = qnn.mbit_encoder_backward(torch.from_numpy(xr).to(dev), torch.from_numpy(gc).to(dev), bits, r).cpu().numpy()
        bound = sum(np.abs(gc[m - 1]).astype(np.float64) * (A / 2 ** m) * math.pi * (math.pi * A / 2 ** m + 8)
                    for m in range(1, bits + 1)) * 2.0 ** -24 / r
        assert np.all(np.abs(got.astype(np.float64) - want) <= bound + 1e-30)
        outside = np.abs((xr / np.float32(r)).astype(np.float32)) > 1
        assert np.all(got[outside] == 0.0)


@pytest.mark.parametrize("bits", [1, 2, 5, 8])
@pytest.mark.parametrize("n", [4, 1024, 262144 + 4, 262144 + 3])
def test_vector_and_scalar_paths_agree_with_oracle(bits, n):
    """n a multiple of 4 takes the float4 kernels, any other n the scalar ones; an offset view breaks the 16-byte
    alignment and must fall back to the scalar path with the same results."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(1000 * bits + n % 997)
    x = rng.uniform(-1.1, 1.1, size=n + 1).astype(np.float32)
    gc = rng.standard_normal((bits, n)).astype(np.float32)
    xd = torch.from_numpy(x).to(dev)
    A = 2 ** bits - 1
    for view, xs in ((xd[:n], x[:n]), (xd[1:], x[1:])):
        got = qnn.mbit_encoder_forward(view, bits, 1.0).cpu().numpy()
        assert np.array_equal(got, oracle.mbit_encoder_forward(xs, bits, 1.0))
        gb = qnn.mbit_encoder_backward(view, torch.from_numpy(gc).to(dev), bits, 1.0).cpu().numpy()
        want = oracle.mbit_encoder_backward(xs, gc, bits, 1.0)
        bound = sum(np.abs(gc[m - 1]).astype(np.float64) * (A / 2 ** m) * math.pi * (math.pi * A / 2 ** m + 8)
                    for m in range(1, bits + 1)) * 2.0 ** -24
        assert np.all(np.abs(gb.astype(np.float64) - want) <= bound + 1e-30)

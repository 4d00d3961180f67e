"""The plain fp32 product that the efficiency experiment (Section 5.4, Fig. 7) is measured against.

It is a comparison line, not a step of the method, so it is checked against a binary64 matrix product: every output
within the rounding bound of a k-term fp32 sum of products, ragged sizes on every edge of the launch grid, and the
exact result when all products and partial sums are small integers.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("m,n,k", [(1, 1, 1), (8, 32, 64), (9, 33, 65), (200, 130, 517), (67, 1000, 300)])
def test_naive_sgemm_matches_float64_product(m, n, k):
    import torch
    from paper_2106_09886_b200 import qnn
    rng = np.random.default_rng(m * 7919 + n * 31 + k)
    a = rng.standard_normal((m, k)).astype(np.float32)
    b = rng.standard_normal((k, n)).astype(np.float32)
    dev = torch.device("cuda:0")
    c = qnn.probe_naive_sgemm(torch.from_numpy(a).to(dev), torch.from_numpy(b).to(dev)).cpu().numpy()
    want = a.astype(np.float64) @ b.astype(np.float64)
    bound = (k + 1) * 2.0 ** -24 * (np.abs(a).astype(np.float64) @ np.abs(b).astype(np.float64)) + 1e-30
    assert np.all(np.abs(c - want) <= bound)


def test_naive_sgemm_is_exact_on_small_integers_and_leaves_neighbours_alone():
    import torch
    from paper_2106_09886_b200 import qnn
    rng = np.random.default_rng(5)
    m, n, k = 37, 45, 900
    a = rng.integers(-7, 8, size=(m, k)).astype(np.float32)
    b = rng.integers(-7, 8, size=(k, n)).astype(np.float32)
    dev = torch.device("cuda:0")
    buf = torch.full((m + 2, n), 123.0, dtype=torch.float32, device=dev)
    qnn.probe_naive_sgemm(torch.from_numpy(a).to(dev), torch.from_numpy(b).to(dev), buf[1:m + 1])
    got = buf.cpu().numpy()
    assert np.array_equal(got[1:m + 1].astype(np.int64), a.astype(np.int64) @ b.astype(np.int64))
    assert np.all(got[0] == 123.0) and np.all(got[m + 1] == 123.0)

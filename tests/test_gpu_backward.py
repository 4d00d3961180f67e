"""GPU parity of the backward products of Algorithm 1 (TF32 tensor-core contractions) against the CPU oracle.

Tolerance.  The codes are exact in TF32 and the accumulator is fp32; each element of g enters with 11 significant
bits (relative error <= 2^-10 whether the hardware truncates or rounds), and a sum of L fp32 terms accumulated in any
order with truncation is off by at most L * 2^-24 relative to the sum of magnitudes.  Hence, element by element,
    |got - want| <= alpha * sum |g| * |q| * (2^-10 + L * 2^-24)     (+ one rounding of the result),
and a g with few significant bits and small integer sums is contracted exactly: those cases are compared with ==."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu


def _codes(rng, rows, k, bits):
    return (2 * rng.integers(0, 2 ** bits, size=(rows, k)) - (2 ** bits - 1)).astype(np.int16)


def _planes_dev(q, bits, dev):
    import torch
    return torch.from_numpy(oracle.pack_planes(q, bits).view(np.int32)).to(dev)


def _bound(g, q_abs_t, alpha, L):
    """alpha * (|g| @ |q|) * (2^-10 + L * 2^-24) for g [rows, L] and q_abs_t [L, cols]."""
    return abs(alpha) * (np.abs(g).astype(np.float64) @ q_abs_t.astype(np.float64)) * (2.0 ** -10 + L * 2.0 ** -24)


@pytest.mark.parametrize("rows,k,bits", [(1, 1, 1), (33, 70, 2), (100, 129, 3), (257, 64, 8), (64, 300, 5)])
def test_unpack_codes_exact(rows, k, bits):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    q = _codes(np.random.default_rng(rows + k), rows, k, bits)
    planes = _planes_dev(q, bits, dev)
    assert np.array_equal(qnn.unpack_codes_f32(planes, rows, k, bits).cpu().numpy(), q.astype(np.float32))
    assert np.array_equal(qnn.unpack_codes_f32(planes, rows, k, bits, transpose=True).cpu().numpy(), q.T.astype(np.float32))


SHAPES = [(128, 128, 128), (5, 8, 3), (130, 260, 200), (257, 100, 129), (64, 36, 1000), (300, 1028, 77), (1, 4, 1),
          (200, 130, 96)]   # (m, n, k); n = 130 takes the padded copy of g


@pytest.mark.parametrize("m,n,k", SHAPES)
@pytest.mark.parametrize("wb", [1, 2, 8])
def test_backward_data_exact_on_integer_gradients(m, n, k, wb):
    """g in {-8..8} and alpha = 1/4: every product and partial sum is an integer below 2^24, so the tensor-core result
    must equal the oracle exactly, whatever the order of accumulation."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(m * 7 + n * 3 + k + wb)
    qw = _codes(rng, n, k, wb)
    g = rng.integers(-8, 9, size=(m, n)).astype(np.float32)
    want = oracle.fc_backward_data(g, qw, 1, wb, 0.25)[0]
    got = qnn.bgemm_backward_data(torch.from_numpy(g).to(dev), _planes_dev(qw, wb, dev), k, wb, 0.25).cpu().numpy()
    assert qnn.tensor_path_status() == 0
    assert np.array_equal(got.astype(np.float64), want)


@pytest.mark.parametrize("m,n,k", SHAPES)
@pytest.mark.parametrize("ab", [1, 2, 8])
def test_backward_weights_exact_on_integer_gradients(m, n, k, ab):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(m * 5 + n * 11 + k + ab)
    qa = _codes(rng, m, k, ab)
    g = rng.integers(-8, 9, size=(m, n)).astype(np.float32)
    want = oracle.fc_backward_weights(g, qa, ab, 1, 0.25)[0]
    got = qnn.bgemm_backward_weights(torch.from_numpy(g).to(dev), _planes_dev(qa, ab, dev), k, ab, 0.25).cpu().numpy()
    assert qnn.tensor_path_status() == 0
    assert np.array_equal(got.astype(np.float64), want)


@pytest.mark.parametrize("m,n,k,ab,wb", [(130, 260, 200, 2, 2), (257, 512, 129, 4, 3), (96, 2048, 64, 8, 8)])
def test_backward_products_within_tf32_bound(m, n, k, ab, wb):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(m + n + k)
    qa, qw = _codes(rng, m, k, ab), _codes(rng, n, k, wb)
    g = rng.standard_normal((m, n)).astype(np.float32)
    alpha = 0.8 / ((2 ** ab - 1) * (2 ** wb - 1))
    gd = torch.from_numpy(g).to(dev)
    G = qnn.bgemm_backward_data(gd, _planes_dev(qw, wb, dev), k, wb, alpha).cpu().numpy().astype(np.float64)
    GW = qnn.bgemm_backward_weights(gd, _planes_dev(qa, ab, dev), k, ab, alpha).cpu().numpy().astype(np.float64)
    assert qnn.tensor_path_status() == 0
    ga = oracle.fc_backward_data(g, qw, ab, wb, alpha)
    gw = oracle.fc_backward_weights(g, qa, ab, wb, alpha)
    bd = _bound(g, np.abs(qw), np.float32(alpha), n)
    bw = _bound(g.T, np.abs(qa), np.float32(alpha), m)
    for p in range(ab):     # g_{a^p} = 2^(p-1) * G
        assert np.all(np.abs(2.0 ** p * G - ga[p]) <= 2.0 ** p * bd * (1 + 2.0 ** -20) + 1e-30)
    for j in range(wb):
        assert np.all(np.abs(2.0 ** j * GW - gw[j]) <= 2.0 ** j * bw * (1 + 2.0 ** -20) + 1e-30)
    # the errors behave like independent roundings: their RMS is far below the worst-case bound
    assert np.sqrt(np.mean((G - ga[0]) ** 2)) <= 0.1 * np.sqrt(np.mean(bd ** 2))
    assert np.sqrt(np.mean((GW - gw[0]) ** 2)) <= 0.1 * np.sqrt(np.mean(bw ** 2))


@pytest.mark.parametrize("m,n,k,ab,wb", [(130, 64, 200, 2, 2), (100, 128, 129, 4, 1), (64, 32, 95, 1, 3)])
def test_backward_data_through_the_encoder(m, n, k, ab, wb):
    """With x given the kernel applies Eq. 12 to gc_p = 2^(p-1) * G in its epilogue: compared with the two oracle
    steps chained (products in binary64, then the encoder derivative)."""
    import math
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(m * n + k)
    qw = _codes(rng, n, k, wb)
    r = 1.7
    x = (rng.uniform(-1.15, 1.15, size=(m, k)) * r).astype(np.float32)
    g = rng.integers(-8, 9, size=(m, n)).astype(np.float32)          # exact G: the comparison isolates the epilogue
    alpha = 0.125
    ga = oracle.fc_backward_data(g, qw, ab, wb, alpha)                # [ab, m, k]
    assert np.array_equal(ga.astype(np.float32).astype(np.float64), ga)
    want = oracle.mbit_encoder_backward(x, ga.reshape(ab, -1).astype(np.float32), ab, r).reshape(m, k)
    got = qnn.bgemm_backward_data(torch.from_numpy(g).to(dev), _planes_dev(qw, wb, dev), k, wb, alpha,
                                  x=torch.from_numpy(x).to(dev), ab=ab, r=r).cpu().numpy().astype(np.float64)
    assert qnn.tensor_path_status() == 0
    A = 2 ** ab - 1
    bound = sum(np.abs(ga[p - 1]) * (A / 2 ** p) * math.pi * (math.pi * A / 2 ** p + 8) for p in range(1, ab + 1)) \
        * 2.0 ** -24 / r
    assert np.all(np.abs(got - want) <= bound + 1e-30)
    outside = np.abs((x / np.float32(r)).astype(np.float32)) > 1
    assert outside.any() and np.all(got[outside] == 0.0)


def test_backward_argument_checks():
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    g = torch.zeros((8, 8), device=dev)
    planes = torch.zeros((8, 1, 4), dtype=torch.int32, device=dev)
    small = torch.empty(16, dtype=torch.uint8, device=dev)
    with pytest.raises(qnn.QnnError) as e:
        qnn.bgemm_backward_data(g, planes, 8, 1, 1.0, workspace=small)
    assert e.value.status == qnn.lib.qnn_bgemm_backward_data(None, None, 0, 0, 0, 1, 1.0, None, 1, 1.0, None, None, 0, None)
    with pytest.raises(qnn.QnnError):
        qnn.bgemm_backward_weights(g, planes, 8, 9, 1.0)
    assert qnn.lib.qnn_bgemm_backward_data_workspace(0, 1, 1) == 0


@pytest.mark.parametrize("m,n,k,ab,wb", [(4096, 4096, 4096, 2, 2), (3000, 4100, 2050, 3, 4)])
def test_backward_products_full_size_sampled(m, n, k, ab, wb):
    """The benchmarked size (and a ragged large one) in the launch configuration run_case.py times: 128 x 256 tiles,
    persistent CTAs.  Sampled outputs against the oracle: exact for integer gradients, within the bound for real ones."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(m + k)
    qa, qw = _codes(rng, m, k, ab), _codes(rng, n, k, wb)
    pa, pw = _planes_dev(qa, ab, dev), _planes_dev(qw, wb, dev)
    count = 300
    r_d, c_d = rng.integers(0, m, count), rng.integers(0, k, count)
    r_w, c_w = rng.integers(0, n, count), rng.integers(0, k, count)
    r_d[:4], c_d[:4] = [0, m - 1, 0, m - 1], [0, k - 1, k - 1, 0]          # tile corners
    r_w[:4], c_w[:4] = [0, n - 1, 0, n - 1], [0, k - 1, k - 1, 0]
    for kind in ("integer", "real"):
        if kind == "integer":
            g, alpha = rng.integers(-8, 9, size=(m, n)).astype(np.float32), 0.25
        else:
            g, alpha = rng.standard_normal((m, n)).astype(np.float32), 0.8 / ((2 ** ab - 1) * (2 ** wb - 1))
        gd = torch.from_numpy(g).to(dev)
        G = qnn.bgemm_backward_data(gd, pw, k, wb, alpha).cpu().numpy().astype(np.float64)
        GW = qnn.bgemm_backward_weights(gd, pa, k, ab, alpha).cpu().numpy().astype(np.float64)
        assert qnn.tensor_path_status() == 0
        want_d = oracle.fc_backward_data_sampled(g, qw, ab, wb, alpha, r_d, c_d)[0]
        want_w = oracle.fc_backward_weights_sampled(g, qa, ab, wb, alpha, r_w, c_w)[0]
        if kind == "integer":
            assert np.array_equal(G[r_d, c_d], want_d) and np.array_equal(GW[r_w, c_w], want_w)
        else:
            a32 = float(np.float32(alpha))
            bd = a32 * np.einsum("in,ni->i", np.abs(g[r_d]).astype(np.float64), np.abs(qw[:, c_d]).astype(np.float64)) \
                * (2.0 ** -10 + n * 2.0 ** -24)
            bw = a32 * np.einsum("ri,ri->i", np.abs(g[:, r_w]).astype(np.float64), np.abs(qa[:, c_w]).astype(np.float64)) \
                * (2.0 ** -10 + m * 2.0 ** -24)
            assert np.all(np.abs(G[r_d, c_d] - want_d) <= bd) and np.all(np.abs(GW[r_w, c_w] - want_w) <= bw)
            # every element is finite and the matrix has the scale the samples have (nothing left unwritten)
            assert np.isfinite(G).all() and np.isfinite(GW).all()
            assert 0.5 < np.std(G) / np.std(want_d) < 2.0 and 0.5 < np.std(GW) / np.std(want_w) < 2.0

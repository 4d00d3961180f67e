"""GPU parity: qnn_encode_pack / qnn_pack_weights / qnn_absmax_f32 against the CPU oracle, bit for bit."""
import numpy as np
import pytest

import oracle
from helpers import oracle_weight_planes

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2106_09886_b200 import qnn
    return torch, qnn, torch.device("cuda:0")


def special_values(scale, bits):
    A = 2 ** bits - 1
    ties = np.arange(-A - 3, A + 4, dtype=np.float64) * float(scale)         # every grid point and every tie
    extra = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 1e-30, -1e-30, 1e30, -1e30, 3.4e38], dtype=np.float64)
    v = np.concatenate([ties, np.nextafter(ties, np.inf), np.nextafter(ties, -np.inf), extra]).astype(np.float32)
    return np.concatenate([v, np.nextafter(v, np.float32(np.inf)), np.nextafter(v, np.float32(-np.inf))])


@pytest.mark.parametrize("bits", range(1, 9))
@pytest.mark.parametrize("rows,k,ldx", [(1, 1, 1), (3, 31, 31), (5, 33, 40), (7, 127, 127), (2, 129, 129), (6, 5, 12), (4, 20, 21),
                                        (300, 3, 3), (9, 50, 51),
                                        (9, 300, 333), (4, 1000, 1000), (33, 512, 512)])
def test_encode_pack_bit_exact(env, bits, rows, k, ldx):
    torch, qnn, dev = env
    rng = np.random.default_rng(bits * 1000 + rows * 10 + k)
    scale = np.float32(0.37) if bits % 2 else np.float32(0.25)
    x = (rng.standard_normal((rows, ldx)) * 2.0 * (2 ** bits - 1) * float(scale) / 3).astype(np.float32)
    sp = special_values(scale, bits)
    flat = x.reshape(-1)
    n = min(flat.size, sp.size)
    flat[:n] = sp[rng.permutation(sp.size)[:n]]
    for relu in (False, True):
        want = oracle.pack_planes(oracle.quantize(x[:, :k], bits, scale, relu), bits)
        t = (oracle.quantize(x[:, :k], bits, scale, relu).astype(np.int64) + 2 ** bits - 1) // 2
        x_d = torch.from_numpy(x).to(dev)
        rowsum = torch.full((rows,), -7, dtype=torch.int32, device=dev)
        planes = torch.full((rows, bits, qnn.row_words(k)), -1, dtype=torch.int32, device=dev)
        qnn.encode_pack(x_d, bits, scale, qnn.RELU if relu else 0, planes=planes, rowsum=rowsum, k=k)
        torch.cuda.synchronize()
        got = planes.cpu().numpy().view(np.uint32)
        assert np.array_equal(got, want)
        assert np.array_equal(rowsum.cpu().numpy(), t.sum(axis=1))
        # without the row sums (the kernels take a different code path for 1 and 2 bits then), and from a
        # source that is only 4-byte aligned (no 16-byte vector loads)
        planes.fill_(-1)
        qnn.encode_pack(x_d, bits, scale, qnn.RELU if relu else 0, planes=planes, k=k)
        assert np.array_equal(planes.cpu().numpy().view(np.uint32), want)
        shifted = torch.empty(x_d.numel() + 1, dtype=torch.float32, device=dev)[1:].view(rows, ldx)
        shifted.copy_(x_d)
        planes.fill_(-1)
        qnn.encode_pack(shifted, bits, scale, qnn.RELU if relu else 0, planes=planes, k=k)
        assert np.array_equal(planes.cpu().numpy().view(np.uint32), want)


def test_encode_pack_all_special_values_every_width(env):
    torch, qnn, dev = env
    for bits in range(1, 9):
        for scale in (np.float32(1.0) / np.float32(3.0), np.float32(0.013), np.float32(2.0)):
            x = special_values(scale, bits).reshape(1, -1)
            want = oracle.pack_planes(oracle.quantize(x, bits, scale), bits)
            got = qnn.encode_pack(torch.from_numpy(x).to(dev), bits, scale).cpu().numpy().view(np.uint32)
            assert np.array_equal(got, want), (bits, scale)


def test_encode_pack_large_ragged(env):
    torch, qnn, dev = env
    rng = np.random.default_rng(0)
    x = np.maximum(rng.standard_normal((1537, 4097)), 0).astype(np.float32)
    scale = np.float32(np.abs(x).max()) / np.float32(7)
    want = oracle.pack_planes(oracle.quantize(x, 3, scale), 3)
    got = qnn.encode_pack(torch.from_numpy(x).to(dev), 3, scale).cpu().numpy().view(np.uint32)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("n_out,taps,c", [(5, 1, 40), (16, 1, 512), (7, 9, 3), (8, 9, 64), (6, 9, 100), (4, 1, 129),
                                          (3, 25, 33), (64, 9, 256)])
def test_pack_weights_all_layouts(env, bits, n_out, taps, c):
    torch, qnn, dev = env
    rng = np.random.default_rng(bits + n_out * 7 + taps * 13 + c)
    w = (0.05 * rng.standard_normal((n_out, taps, c))).astype(np.float32)
    scale = np.float32(np.abs(w).max()) / np.float32(2 ** bits - 1)
    want_planes, want_tapsum = oracle_weight_planes(oracle.quantize(w, bits, scale), bits)
    views = {qnn.W_NTC: w, qnn.W_TCN: np.ascontiguousarray(w.transpose(1, 2, 0)),
             qnn.W_NCT: np.ascontiguousarray(w.transpose(0, 2, 1))}
    for layout, arr in views.items():
        packed = qnn.pack_weights(torch.from_numpy(arr).to(dev), n_out, taps, c, layout, bits, scale)
        planes, tapsum = qnn.weights_views(packed, n_out, taps, c, bits)
        torch.cuda.synchronize()
        assert np.array_equal(planes.cpu().numpy().view(np.uint32), want_planes), layout
        assert np.array_equal(tapsum.cpu().numpy(), want_tapsum), layout


def test_absmax(env):
    torch, qnn, dev = env
    rng = np.random.default_rng(4)
    for n in [1, 31, 1000, 1 << 20]:
        x = rng.standard_normal(n).astype(np.float32)
        x[rng.integers(0, n)] = np.float32(-17.25)
        if n > 10:
            x[3] = np.nan
        got = qnn.absmax_f32(torch.from_numpy(x).to(dev)).cpu().numpy()[0]
        assert got == np.float32(17.25)


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("rows,k", [(1, 3), (7, 3), (1001, 3), (5, 32), (1000, 32), (3, 33), (999, 64), (1234, 40),
                                    (6, 65), (4097, 64), (50000, 16)])
def test_encode_pack_short_rows(env, bits, rows, k):
    """Rows of at most 64 elements (NHWC activations with few channels) take the multi-row path."""
    torch, qnn, dev = env
    rng = np.random.default_rng(bits * 100 + rows + k)
    x = rng.standard_normal((rows, k)).astype(np.float32)
    scale = np.float32(np.abs(x).max()) / np.float32(2 ** bits - 1)
    for relu in (False, True):
        q = oracle.quantize(x, bits, scale, relu)
        want = oracle.pack_planes(q, bits)
        rowsum = torch.full((rows,), -7, dtype=torch.int32, device=dev)
        got = qnn.encode_pack(torch.from_numpy(x).to(dev), bits, scale, qnn.RELU if relu else 0, rowsum=rowsum)
        torch.cuda.synchronize()
        assert np.array_equal(got.cpu().numpy().view(np.uint32), want)
        assert np.array_equal(rowsum.cpu().numpy(), ((q.astype(np.int64) + 2 ** bits - 1) // 2).sum(axis=1))

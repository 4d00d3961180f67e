"""GPU parity for layers whose whole reduction is at most four words per plane (Kg <= 128): fully-connected layers
with short rows and 1x1 convolutions without padding (the stride-2 projections of a residual network).  They run on
a kernel of their own that compresses the xor words of ALL plane pairs of an output through full adders before
counting; every (ab, wb) in 1..4 x 1..4 with 1 to 4 words per plane is a separate instantiation, so each is checked
here, together with ragged rows and features, strides, a padded leading dimension and the extreme codes."""
import numpy as np
import pytest

from helpers import assert_fp32_close, gpu_conv, gpu_fc, oracle_conv, oracle_fc, scales_for

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("ab", [1, 2, 3, 4])
@pytest.mark.parametrize("wb", [1, 2, 3, 4])
def test_fc_short_rows_every_instantiation(ab, wb):
    rng = np.random.default_rng(ab * 10 + wb)
    for Kg in (7, 32, 33, 64, 90, 96, 127, 128):                       # 1, 1, 2, 2, 3, 3, 4, 4 words per plane
        Mg, Ng = int(rng.integers(1, 150)), int(rng.integers(1, 200))
        a = rng.standard_normal((Mg, Kg)).astype(np.float32)
        w = rng.standard_normal((Ng, Kg)).astype(np.float32)
        sa, sw, alpha = scales_for(a, w, ab, wb)
        _, _, acc, out = oracle_fc(a, w, False, ab, wb, sa, sw, alpha)
        got = gpu_fc(a, w, False, ab, wb, sa, sw, alpha)
        assert np.array_equal(got["acc"], acc), (Mg, Ng, Kg)
        assert_fp32_close(got["out"], out)


@pytest.mark.parametrize("ab,wb", [(1, 1), (2, 2), (3, 3), (4, 4), (4, 1), (2, 3)])
def test_fc_short_rows_extreme_codes(ab, wb):
    """All codes at the ends of the range: every xor word is all ones or all zeros, so every carry chain of the
    adder tree is exercised at full length."""
    A, B = 2 ** ab - 1, 2 ** wb - 1
    for Kg in (32, 64, 96, 128, 100):
        a = np.full((40, Kg), 1e6, np.float32)
        w = np.full((70, Kg), 1e6, np.float32)
        one = np.float32(1)
        assert np.all(gpu_fc(a, w, False, ab, wb, one, one, one)["acc"] == Kg * A * B)
        assert np.all(gpu_fc(a, -w, False, ab, wb, one, one, one)["acc"] == -Kg * A * B)
        w[::2] *= -1
        got = gpu_fc(-a, w, False, ab, wb, one, one, one)["acc"]
        assert np.all(got[:, ::2] == Kg * A * B) and np.all(got[:, 1::2] == -Kg * A * B)


@pytest.mark.parametrize("N,H,W,C,Cout,stride,ab,wb", [
    (2, 8, 8, 64, 128, 2, 3, 3), (2, 7, 9, 128, 256, 2, 3, 3), (1, 5, 5, 32, 33, 1, 2, 2), (3, 6, 4, 96, 70, 3, 4, 4),
    (2, 9, 9, 100, 40, 2, 1, 3), (1, 12, 12, 64, 64, 1, 4, 2), (5, 3, 3, 33, 300, 2, 2, 4)])
def test_pointwise_convolutions(N, H, W, C, Cout, stride, ab, wb):
    rng = np.random.default_rng(N * 1000 + H * 100 + C + Cout)
    a = np.maximum(rng.standard_normal((N, H, W, C)), 0).astype(np.float32)
    w = (0.05 * rng.standard_normal((Cout, 1, 1, C))).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_conv(a, w, ab, wb, sa, sw, alpha, stride, 0)
    got = gpu_conv(a, w, ab, wb, sa, sw, alpha, stride, 0)
    assert np.array_equal(got["acc"], acc)
    assert_fp32_close(got["out"], out)


def test_fc_short_rows_padded_leading_dimension_and_single_outputs():
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(5)
    Mg, Ng, Kg, ab, wb = 77, 45, 100, 3, 2
    a = rng.standard_normal((Mg, Kg)).astype(np.float32)
    w = rng.standard_normal((Ng, Kg)).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_fc(a, w, False, ab, wb, sa, sw, alpha)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev), ab, sa)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Ng, 1, Kg, qnn.W_NTC, wb, sw)
    wide = torch.full((Mg, Ng + 11), -3.0, dtype=torch.float32, device=dev)
    qnn.bgemm(planes, ab, packed, wb, Mg, Ng, Kg, alpha, out=wide[:, :Ng])
    assert_fp32_close(wide[:, :Ng].cpu().numpy(), out)
    assert torch.all(wide[:, Ng:] == -3.0)
    acc_d = torch.empty((Mg, Ng), dtype=torch.int32, device=dev)
    assert qnn.lib.qnn_bgemm(planes.data_ptr(), ab, packed.data_ptr(), wb, Mg, Ng, Kg, float(alpha), None, Ng,
                             acc_d.data_ptr(), None) == 0
    torch.cuda.synchronize()
    assert np.array_equal(acc_d.cpu().numpy(), acc)


@pytest.mark.parametrize("Mg,Ng,Kg,ab,wb,nb", [(70, 17, 64, 3, 3, 3), (33, 130, 96, 1, 1, 1), (200, 64, 128, 4, 4, 4),
                                               (45, 100, 33, 2, 3, 8), (129, 257, 100, 3, 2, 2)])
def test_fc_short_rows_chained(Mg, Ng, Kg, ab, wb, nb):
    """The chaining epilogue of the short-reduction kernel: next-layer planes (code bytes gathered into words per row,
    padding words cleared) bit-identical to the oracle's quantize + pack of the oracle's fp32 result, with and
    without the fp32 output, with and without the per-feature affine."""
    import torch
    import oracle
    from paper_2106_09886_b200 import qnn
    from paper_2106_09886_b200 import workloads as wl
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(Mg + 7 * Ng + Kg)
    a = rng.standard_normal((Mg, Kg)).astype(np.float32)
    w = rng.standard_normal((Ng, Kg)).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_fc(a, w, False, ab, wb, sa, sw, alpha)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev), ab, sa)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Ng, 1, Kg, qnn.W_NTC, wb, sw)
    gamma = rng.standard_normal(Ng).astype(np.float32)
    beta = rng.standard_normal(Ng).astype(np.float32)
    for affine in (False, True):
        y = oracle.affine(out, gamma, beta) if affine else out
        for relu in (True, False):
            ns = wl.per_tensor_scale(np.maximum(y, 0) if relu else y, nb)
            want = oracle.pack_planes(oracle.quantize(y, nb, ns, relu), nb)
            for with_out in (False, True):
                nxt = torch.full((Mg, nb, qnn.row_words(Ng)), -1, dtype=torch.int32, device=dev)
                out_d = torch.full((Mg, Ng), 7.0, dtype=torch.float32, device=dev) if with_out else None
                kw = dict(ch_gamma=torch.from_numpy(gamma).to(dev), ch_beta=torch.from_numpy(beta).to(dev)) if affine else {}
                qnn.bgemm_encode(planes, ab, packed, wb, Mg, Ng, Kg, alpha, nb, ns, qnn.RELU if relu else 0,
                                 next_planes=nxt, out=out_d, **kw)
                torch.cuda.synchronize()
                assert np.array_equal(nxt.cpu().numpy().view(np.uint32), want)
                if with_out:
                    assert np.array_equal(out_d.cpu().numpy(), y) if affine else True
                    assert_fp32_close(out_d.cpu().numpy(), y)


@pytest.mark.parametrize("N,H,W,C,Cout,stride,ab,wb,nb", [(2, 8, 8, 64, 128, 2, 3, 3, 3), (1, 9, 7, 128, 70, 2, 3, 3, 3),
                                                         (3, 5, 5, 96, 33, 1, 2, 4, 5)])
def test_pointwise_convolutions_chained(N, H, W, C, Cout, stride, ab, wb, nb):
    import torch
    import oracle
    from paper_2106_09886_b200 import qnn
    from paper_2106_09886_b200 import workloads as wl
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(N * 100 + H + C + Cout)
    a = rng.standard_normal((N, H, W, C)).astype(np.float32)
    w = (0.05 * rng.standard_normal((Cout, 1, 1, C))).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_conv(a, w, ab, wb, sa, sw, alpha, stride, 0, relu=True)
    ns = wl.per_tensor_scale(np.maximum(out, 0), nb)
    want = oracle.pack_planes(oracle.quantize(out.reshape(-1, Cout), nb, ns, True), nb)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev).view(-1, C), ab, sa, qnn.RELU)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Cout, 1, C, qnn.W_NTC, wb, sw)
    Mg = out.shape[0] * out.shape[1] * out.shape[2]
    for with_out in (False, True):
        nxt = torch.full((Mg, nb, qnn.row_words(Cout)), -1, dtype=torch.int32, device=dev)
        out_d = torch.empty(out.shape, dtype=torch.float32, device=dev) if with_out else None
        qnn.bconv2d_encode(planes, ab, packed, wb, N, H, W, C, Cout, 1, 1, stride, 0, alpha, nb, ns, qnn.RELU,
                           next_planes=nxt, out=out_d)
        torch.cuda.synchronize()
        assert np.array_equal(nxt.cpu().numpy().view(np.uint32), want)
        if with_out:
            assert_fp32_close(out_d.cpu().numpy(), out)

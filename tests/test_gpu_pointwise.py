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

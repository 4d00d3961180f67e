"""GPU parity on mid-sized layers: a few to a few hundred output tiles with long reductions.

These are the shapes between the small cases (one tile or two) and the full-size configurations: the last round of
output tiles is partly filled, reductions run over 4 to 16 stages and end in padded groups or short tails, rows and
columns are ragged, and each of the two outputs (fp32 result, int32 accumulators) is also requested alone, the fp32
one with a padded leading dimension.  Accumulators must be bit-exact, outputs within 1e-6 relative.
"""
import numpy as np
import pytest

from helpers import assert_fp32_close, gpu_conv, gpu_fc, oracle_conv, oracle_fc, scales_for

pytestmark = pytest.mark.gpu


# (Mg, Ng, Kg, ab, wb): output tiles are 64 or 32 rows x 64 features, a stage is 512 elements of the reduction
# (296 tiles = two per SM on 148 SMs)
FC_CASES = [
    (640, 640, 2048, 2, 2),      # 100 tiles of 64 rows, 4 stages
    (320, 320, 2048, 2, 2),      # a few dozen tiles
    (130, 70, 2088, 2, 2),       # ragged rows and columns, 5 stages ending in a zero-padded group
    (200, 100, 8192, 1, 1),      # a handful of tiles, 16 stages
    (200, 100, 8192 + 70, 2, 1), # the same with a tail of three words after the full groups
    (150, 512, 3000, 3, 3),      # 32-row tiles (5 x 8), 6 stages
    (97, 129, 4096, 4, 2),       # 4 x 3 tiles, 8 stages
    (64 * 20, 64 * 20, 2048, 2, 2),   # 400 tiles = one full round of 296 + 104 left over
    (64 * 37, 64 * 9, 2560, 2, 2),    # 333 tiles = 296 + 37: a few dozen tiles behind a full round
    (32 * 30, 64 * 10, 2100, 3, 2),   # 300 tiles = 296 + 4, 32-row tiles
]


@pytest.mark.parametrize("Mg,Ng,Kg,ab,wb", FC_CASES)
def test_fc_midsize(Mg, Ng, Kg, ab, wb):
    rng = np.random.default_rng(Mg * 31 + Ng * 7 + Kg + ab)
    a = rng.standard_normal((Mg, Kg)).astype(np.float32)
    w = rng.standard_normal((Ng, Kg)).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_fc(a, w, False, ab, wb, sa, sw, alpha)
    got = gpu_fc(a, w, False, ab, wb, sa, sw, alpha)
    assert np.array_equal(got["acc"], acc)
    assert_fp32_close(got["out"], out)
    # fp32 output alone (with a padded leading dimension), and accumulators alone
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev), ab, sa)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Ng, 1, Kg, qnn.W_NTC, wb, sw)
    wide = torch.full((Mg, Ng + 5), 7.0, dtype=torch.float32, device=dev)
    qnn.bgemm(planes, ab, packed, wb, Mg, Ng, Kg, alpha, out=wide[:, :Ng])
    assert_fp32_close(wide[:, :Ng].cpu().numpy(), out)
    assert torch.all(wide[:, Ng:] == 7.0)
    acc_d = torch.full((Mg, Ng), 12345, dtype=torch.int32, device=dev)
    assert qnn.lib.qnn_bgemm(planes.data_ptr(), ab, packed.data_ptr(), wb, Mg, Ng, Kg, float(alpha), None, Ng,
                             acc_d.data_ptr(), None) == 0
    torch.cuda.synchronize()
    assert np.array_equal(acc_d.cpu().numpy(), acc)


# (N, H, W, C, Cout, stride, pad, ab, wb), 3 x 3 kernels: 9 * ceil(C/32) words per plane
CONV_CASES = [
    (3, 14, 14, 256, 256, 1, 1, 2, 2),     # a few dozen tiles, 5 stages
    (32, 14, 14, 256, 256, 1, 1, 2, 2),    # the single-convolution configuration: 392 tiles = 296 + 96
    (2, 7, 7, 512, 130, 1, 1, 3, 3),       # 4 x 3 tiles, 9 stages
    (5, 9, 9, 200, 70, 2, 1, 4, 4),        # strided, ragged channel words (7 per tap, 4-byte copies)
    (1, 20, 20, 160, 64, 1, 0, 1, 2),      # no padding, 1-bit activations
]


@pytest.mark.parametrize("N,H,W,C,Cout,stride,pad,ab,wb", CONV_CASES)
def test_conv_midsize(N, H, W, C, Cout, stride, pad, ab, wb):
    rng = np.random.default_rng(N * 1000 + H * 100 + C + Cout)
    a = np.maximum(rng.standard_normal((N, H, W, C)), 0).astype(np.float32)
    w = (0.02 * rng.standard_normal((Cout, 3, 3, C))).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    _, _, acc, out = oracle_conv(a, w, ab, wb, sa, sw, alpha, stride, pad)
    got = gpu_conv(a, w, ab, wb, sa, sw, alpha, stride, pad)
    assert np.array_equal(got["acc"], acc)
    assert_fp32_close(got["out"], out)
    again = gpu_conv(a, w, ab, wb, sa, sw, alpha, stride, pad)
    assert np.array_equal(again["acc"], got["acc"])             # repeatable bit for bit

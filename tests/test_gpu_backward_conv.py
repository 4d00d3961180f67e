"""GPU parity of the backward products of a convolution layer (Algorithm 1 backward; TF32 tensor-core contractions:
the data gradient as an implicit GEMM whose operand the TMA unit gathers from the gradient image, the weight gradient
on staged activation codes) against the CPU oracle.

Tolerance, element by element, as for the fully-connected products:
    |got - want| <= alpha * sum |g| * |q| * (2^-10 + L * 2^-24)
over the terms of that element's sum, with L the contraction length on the tensor cores (R*S*Cout for the data
gradient: taps and output features are one accumulation; N*Ho*Wo for the weight gradient).
Integer-valued g with alpha a power of two is contracted exactly and compared with ==, which pins every index of the
gather (stride classes, tap shifts, zero fill outside the gradient image), of the tap-major weight layout and of the
tile-row-to-pixel mapping independently of rounding."""
import numpy as np
import pytest

import oracle
from helpers import oracle_weight_planes

pytestmark = pytest.mark.gpu

# (N, H, W, C, Cout, R, S, stride, pad): ragged channel counts, strides, 1x1, a 5x5, Cout % 4 != 0 (padded copy of g)
GEOMS = [(2, 6, 5, 3, 4, 3, 3, 1, 1), (1, 9, 9, 40, 6, 3, 3, 2, 1), (3, 8, 8, 64, 16, 1, 1, 2, 0), (2, 7, 6, 33, 5, 5, 5, 1, 2),
         (2, 14, 14, 128, 32, 3, 3, 1, 1), (1, 5, 4, 70, 130, 3, 2, 1, 0), (5, 12, 12, 16, 24, 3, 3, 2, 2),
         # stride 3 with a 5 x 4 kernel (nine stride classes with different tap sets), a wide image (several tiles along
         # w), many images of 7 x 7 (tiles that span images), more than 256 channels (several channel tiles)
         (2, 11, 10, 8, 12, 5, 4, 3, 2), (1, 3, 150, 16, 8, 3, 3, 1, 1), (37, 7, 7, 24, 40, 3, 3, 1, 1), (2, 6, 6, 300, 20, 3, 3, 2, 1),
         # a 7 x 7 kernel at stride 2 (a network's stem): the weight gradient's strided copies of the codes, two row parities
         (2, 16, 16, 8, 12, 7, 7, 2, 3),
         # output rows of a multiple of four columns (no row padding: the gradient goes through the plain transpose)
         (3, 8, 8, 20, 12, 3, 3, 1, 1)]


def _codes(rng, shape, bits):
    return (2 * rng.integers(0, 2 ** bits, size=shape) - (2 ** bits - 1)).astype(np.int16)


def _packed_weights_dev(qw, wb, dev):
    """The blob qnn_pack_weights would write for these codes, assembled from the oracle's canonical packer."""
    import torch
    Cout, R, S, C = qw.shape
    planes, tapsum = oracle_weight_planes(qw.reshape(Cout, R * S, C), wb)
    blob = np.concatenate([planes.reshape(-1).view(np.uint8), tapsum.reshape(-1).view(np.uint8)])
    return torch.from_numpy(blob).to(dev)


def _case(seed, geom, ab, wb, integer_g):
    N, H, W, C, Cout, R, S, stride, pad = geom
    rng = np.random.default_rng(seed)
    qa, qw = _codes(rng, (N, H, W, C), ab), _codes(rng, (Cout, R, S, C), wb)
    Ho, Wo = oracle.conv_out_dim(H, R, stride, pad), oracle.conv_out_dim(W, S, stride, pad)
    g = (rng.integers(-8, 9, size=(N, Ho, Wo, Cout)) if integer_g else rng.standard_normal((N, Ho, Wo, Cout))).astype(np.float32)
    return qa, qw, g


@pytest.mark.parametrize("geom", GEOMS)
@pytest.mark.parametrize("wb", [1, 3, 8])
def test_conv_backward_data_exact_on_integer_gradients(geom, wb):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    N, H, W, C, Cout, R, S, stride, pad = geom
    qa, qw, g = _case(sum(geom) + wb, geom, 1, wb, True)
    want = oracle.conv_backward_data(g, qw, (H, W), stride, pad, 1, wb, 0.25)[0]
    got = qnn.bconv2d_backward_data(torch.from_numpy(g).to(dev), _packed_weights_dev(qw, wb, dev), wb, H, W, C, R, S,
                                    stride, pad, 0.25).cpu().numpy()
    assert qnn.tensor_path_status() == 0
    assert np.array_equal(got.astype(np.float64), want)


@pytest.mark.parametrize("geom", GEOMS)
@pytest.mark.parametrize("ab", [1, 2, 8])
def test_conv_backward_weights_exact_on_integer_gradients(geom, ab):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    N, H, W, C, Cout, R, S, stride, pad = geom
    qa, qw, g = _case(sum(geom) * 3 + ab, geom, ab, 1, True)
    want = oracle.conv_backward_weights(g, qa, (R, S), stride, pad, ab, 1, 0.25)[0]
    planes = torch.from_numpy(oracle.pack_planes(qa.reshape(-1, C), ab).view(np.int32)).to(dev)
    got = qnn.bconv2d_backward_weights(torch.from_numpy(g).to(dev), planes, ab, H, W, C, R, S, stride, pad, 0.25).cpu().numpy()
    assert qnn.tensor_path_status() == 0
    assert np.array_equal(got.astype(np.float64), want)


def test_conv_backward_weights_split_contraction_is_exact_and_repeatable():
    """Few output tiles against thousands of output pixels: the contraction is split over many CTAs and the partial
    products are summed in a fixed order, so integer gradients stay exact and two calls agree bit for bit."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    geom, ab = (8, 28, 28, 32, 16, 3, 3, 1, 1), 2
    N, H, W, C, Cout, R, S, stride, pad = geom
    qa, qw, g = _case(77, geom, ab, 1, True)
    want = oracle.conv_backward_weights(g, qa, (R, S), stride, pad, ab, 1, 0.25)[0]
    planes = torch.from_numpy(oracle.pack_planes(qa.reshape(-1, C), ab).view(np.int32)).to(dev)
    gd = torch.from_numpy(g).to(dev)
    got = qnn.bconv2d_backward_weights(gd, planes, ab, H, W, C, R, S, stride, pad, 0.25).cpu().numpy()
    assert qnn.tensor_path_status() == 0
    assert np.array_equal(got.astype(np.float64), want)
    gr = torch.from_numpy(np.random.default_rng(1).standard_normal(g.shape).astype(np.float32)).to(dev)
    a1 = qnn.bconv2d_backward_weights(gr, planes, ab, H, W, C, R, S, stride, pad, 0.37).cpu().numpy()
    a2 = qnn.bconv2d_backward_weights(gr, planes, ab, H, W, C, R, S, stride, pad, 0.37).cpu().numpy()
    assert np.array_equal(a1, a2)


@pytest.mark.parametrize("geom,ab,wb", [((2, 14, 14, 64, 48, 3, 3, 1, 1), 2, 2), ((4, 16, 16, 32, 64, 3, 3, 2, 1), 3, 4),
                                        ((1, 10, 9, 100, 36, 1, 1, 1, 0), 8, 8)])
def test_conv_backward_within_tf32_bound(geom, ab, wb):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    N, H, W, C, Cout, R, S, stride, pad = geom
    qa, qw, g = _case(sum(geom), geom, ab, wb, False)
    alpha = float(np.float32(0.8 / ((2 ** ab - 1) * (2 ** wb - 1))))
    gd = torch.from_numpy(g).to(dev)
    G = qnn.bconv2d_backward_data(gd, _packed_weights_dev(qw, wb, dev), wb, H, W, C, R, S, stride, pad, alpha).cpu().numpy()
    planes = torch.from_numpy(oracle.pack_planes(qa.reshape(-1, C), ab).view(np.int32)).to(dev)
    GW = qnn.bconv2d_backward_weights(gd, planes, ab, H, W, C, R, S, stride, pad, alpha).cpu().numpy()
    assert qnn.tensor_path_status() == 0
    ga = oracle.conv_backward_data(g, qw, (H, W), stride, pad, ab, wb, alpha)
    gw = oracle.conv_backward_weights(g, qa, (R, S), stride, pad, ab, wb, alpha)
    # sums of magnitudes: the same two oracle functions on |g| and on all-(+max) stand-ins are not available for
    # arbitrary codes, so take them from the plain definition with absolute values (1-bit planes of +1 = |q| bound)
    Mg = g.shape[0] * g.shape[1] * g.shape[2]
    mag_d = oracle.conv_backward_data(np.abs(g), np.full_like(qw, 2 ** wb - 1), (H, W), stride, pad, 1, wb, alpha)[0]
    mag_w = oracle.conv_backward_weights(np.abs(g), np.full_like(qa, 2 ** ab - 1), (R, S), stride, pad, ab, 1, alpha)[0]
    bd = mag_d * (2.0 ** -10 + Cout * R * S * 2.0 ** -24)
    bw = mag_w * (2.0 ** -10 + Mg * 2.0 ** -24)
    for p in range(ab):
        assert np.all(np.abs(2.0 ** p * G.astype(np.float64) - ga[p]) <= 2.0 ** p * bd * (1 + 2.0 ** -20) + 1e-30)
    for j in range(wb):
        assert np.all(np.abs(2.0 ** j * GW.astype(np.float64) - gw[j]) <= 2.0 ** j * bw * (1 + 2.0 ** -20) + 1e-30)
    assert np.sqrt(np.mean((G - ga[0]) ** 2)) <= 0.1 * np.sqrt(np.mean(bd ** 2))
    assert np.sqrt(np.mean((GW - gw[0]) ** 2)) <= 0.1 * np.sqrt(np.mean(bw ** 2))


def test_conv_backward_config2_layer_exact():
    """The 3x3, 256 -> 256 channel layer of the single-convolution configuration at 14 x 14 (batch 8 of its 32, which
    the oracle finishes in seconds): many tiles, a ragged last one, 2304-long patches, a split weight contraction."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    geom, ab, wb = (8, 14, 14, 256, 256, 3, 3, 1, 1), 2, 2
    N, H, W, C, Cout, R, S, stride, pad = geom
    qa, qw, g = _case(2, geom, ab, wb, True)
    gd = torch.from_numpy(g).to(dev)
    G = qnn.bconv2d_backward_data(gd, _packed_weights_dev(qw, wb, dev), wb, H, W, C, R, S, stride, pad, 0.125).cpu().numpy()
    planes = torch.from_numpy(oracle.pack_planes(qa.reshape(-1, C), ab).view(np.int32)).to(dev)
    GW = qnn.bconv2d_backward_weights(gd, planes, ab, H, W, C, R, S, stride, pad, 0.125).cpu().numpy()
    assert qnn.tensor_path_status() == 0
    ga = oracle.conv_backward_data(g, qw, (H, W), stride, pad, ab, wb, 0.125)
    gw = oracle.conv_backward_weights(g, qa, (R, S), stride, pad, ab, wb, 0.125)
    for p in range(ab):          # g_{a^p} = 2^(p-1) * G, exactly (integer gradients, sums far below 2^24)
        assert np.array_equal(2.0 ** p * G.astype(np.float64), ga[p])
    for j in range(wb):
        assert np.array_equal(2.0 ** j * GW.astype(np.float64), gw[j])


def test_conv_backward_data_through_the_encoder():
    """With x given the gather applies Eq. 12 to gc_p = 2^(p-1) * G: compared with the oracle's two steps chained."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    geom, ab, wb = (2, 9, 8, 24, 16, 3, 3, 1, 1), 3, 2
    N, H, W, C, Cout, R, S, stride, pad = geom
    qa, qw, g = _case(11, geom, ab, wb, True)
    rng = np.random.default_rng(5)
    x = (rng.random((N, H, W, C)) * 2.4 - 1.2).astype(np.float32)          # some elements outside [-r, r]
    r = 1.0
    got = qnn.bconv2d_backward_data(torch.from_numpy(g).to(dev), _packed_weights_dev(qw, wb, dev), wb, H, W, C, R, S, stride,
                                    pad, 0.25, x=torch.from_numpy(x).to(dev), ab=ab, r=r).cpu().numpy()
    assert qnn.tensor_path_status() == 0
    ga = oracle.conv_backward_data(g, qw, (H, W), stride, pad, ab, wb, 0.25)       # exact here (integer g)
    want = oracle.mbit_encoder_backward(x.reshape(-1), ga.reshape(ab, -1), ab, r).reshape(x.shape)
    # the products are exact; what remains is the binary32 evaluation of Eq. 12 (same bound as the stand-alone kernel)
    k = np.array([(2 ** ab - 1) / 2 ** m for m in range(1, ab + 1)])
    tol = (np.abs(ga).reshape(ab, -1) * (k * np.pi * (np.pi * k + 8))[:, None]).sum(axis=0).reshape(x.shape) * 2.0 ** -24 / r
    assert np.all(np.abs(got - want) <= tol + 1e-30)
    assert np.all(got[np.abs(x) > r] == 0.0)


@pytest.mark.parametrize("geom", [(2, 14, 14, 128, 32, 3, 3, 1, 1), (1, 5, 4, 70, 130, 3, 2, 1, 0), (8, 28, 28, 32, 16, 3, 3, 1, 1)])
def test_conv_backward_stays_inside_its_buffers(geom):
    """Outputs and the workspace (exactly the size the query returns) sit between sentinel regions; nothing outside them
    may change, whichever staging path (padded copy of g, split contraction) the geometry takes."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    N, H, W, C, Cout, R, S, stride, pad = geom
    qa, qw, g = _case(5, geom, 2, 2, True)
    gd = torch.from_numpy(g).to(dev)
    planes = torch.from_numpy(oracle.pack_planes(qa.reshape(-1, C), 2).view(np.int32)).to(dev)
    blob = _packed_weights_dev(qw, 2, dev)
    G = 4096                                                   # guard bytes on each side (keeps 256-byte alignment)

    def guarded(nbytes):
        buf = torch.full((G + nbytes + G,), 0xA5, dtype=torch.uint8, device=dev)
        return buf, buf[G:G + nbytes]

    def intact(buf, nbytes):
        return bool((buf[:G] == 0xA5).all()) and bool((buf[G + nbytes:] == 0xA5).all())

    nd = qnn.lib.qnn_bconv2d_backward_data_workspace(N, H, W, C, Cout, R, S, stride, pad)
    nw = qnn.lib.qnn_bconv2d_backward_weights_workspace(N, H, W, C, Cout, R, S, stride, pad)
    wsd_buf, wsd = guarded(nd)
    wsw_buf, wsw = guarded(nw)
    out_buf, out_b = guarded(N * H * W * C * 4)
    gw_buf, gw_b = guarded(Cout * R * S * C * 4)
    out = out_b.view(torch.float32).view(N, H, W, C)
    gw = gw_b.view(torch.float32).view(Cout, R, S, C)
    qnn.bconv2d_backward_data(gd, blob, 2, H, W, C, R, S, stride, pad, 0.25, out=out, workspace=wsd)
    qnn.bconv2d_backward_weights(gd, planes, 2, H, W, C, R, S, stride, pad, 0.25, gw=gw, workspace=wsw)
    assert qnn.tensor_path_status() == 0
    assert intact(wsd_buf, nd) and intact(wsw_buf, nw) and intact(out_buf, out_b.numel()) and intact(gw_buf, gw_b.numel())
    assert np.array_equal(out.cpu().numpy().astype(np.float64), oracle.conv_backward_data(g, qw, (H, W), stride, pad, 1, 2, 0.25)[0])
    assert np.array_equal(gw.cpu().numpy().astype(np.float64), oracle.conv_backward_weights(g, qa, (R, S), stride, pad, 2, 1, 0.25)[0])


def test_conv_backward_rejects_bad_arguments():
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    g = torch.zeros((1, 4, 4, 8), device=dev)
    assert qnn.lib.qnn_bconv2d_backward_data_workspace(1, 2, 2, 8, 8, 3, 3, 1, 0) == 0          # kernel larger than input
    assert qnn.lib.qnn_bconv2d_backward_weights_workspace(1, 4, 4, 8, 8, 3, 3, 0, 1) == 0        # stride 0
    qw = np.ones((8, 3, 3, 8), dtype=np.int16)
    blob = _packed_weights_dev(qw, 1, dev)
    small = torch.empty(16, dtype=torch.uint8, device=dev)
    with pytest.raises(qnn.QnnError):
        qnn.bconv2d_backward_data(g, blob, 1, 4, 4, 8, 3, 3, 1, 1, 1.0, workspace=small)
    with pytest.raises(qnn.QnnError):
        qnn.bconv2d_backward_data(g, blob, 9, 4, 4, 8, 3, 3, 1, 1, 1.0)

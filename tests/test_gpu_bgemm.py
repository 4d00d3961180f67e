"""GPU parity: qnn_bgemm against the CPU oracle -- int32 accumulators bit-exact, fp32 outputs within 1e-6 relative."""
import numpy as np
import pytest

import oracle
from helpers import assert_fp32_close, gpu_fc, oracle_fc, oracle_fc_codes, scales_for
from paper_2106_09886_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run_case(a, w, k_major, ab, wb, relu=False):
    sa, sw, alpha = scales_for(a, w, ab, wb)
    qa, qw, acc, out = oracle_fc(a, w, k_major, ab, wb, sa, sw, alpha, relu)
    got = gpu_fc(a, w, k_major, ab, wb, sa, sw, alpha, relu, want_planes=True)
    assert np.array_equal(got["a_planes"], oracle.pack_planes(qa, ab))
    assert np.array_equal(got["w_planes"], oracle.pack_planes(qw, wb))
    assert np.array_equal(got["acc"], acc)
    assert_fp32_close(got["out"], out)
    return got


BITS = [(a, w) for a in range(1, 5) for w in range(1, 5)] + [(8, 8), (5, 3), (1, 7), (6, 2)]


@pytest.mark.parametrize("ab,wb", BITS)
def test_bgemm_bit_widths(ab, wb):
    rng = np.random.default_rng(ab * 10 + wb)
    a = np.maximum(rng.standard_normal((150, 700)), 0).astype(np.float32)
    w = (0.02 * rng.standard_normal((83, 700))).astype(np.float32)
    run_case(a, w, False, ab, wb)


@pytest.mark.parametrize("Mg,Ng,Kg", [(1, 1, 1), (1, 5, 31), (63, 17, 32), (64, 64, 128), (65, 100, 129),
                                      (130, 33, 1000), (257, 129, 520), (5, 300, 4097), (200, 8, 96)])
def test_bgemm_ragged_shapes(Mg, Ng, Kg):
    rng = np.random.default_rng(Mg * 7 + Ng * 3 + Kg)
    a = rng.standard_normal((Mg, Kg)).astype(np.float32)
    w = rng.standard_normal((Ng, Kg)).astype(np.float32)
    for ab, wb in [(2, 2), (3, 2)]:
        run_case(a, w, False, ab, wb)


def test_bgemm_closed_forms_and_extremes():
    Kg = 777
    for ab, wb in [(1, 1), (2, 2), (4, 4), (8, 8)]:
        A, B = 2 ** ab - 1, 2 ** wb - 1
        a = np.full((70, Kg), 1e6, np.float32)         # far outside the range: end codes
        w = np.full((66, Kg), 1e6, np.float32)
        got = gpu_fc(a, w, False, ab, wb, np.float32(1), np.float32(1), np.float32(1))
        assert np.all(got["acc"] == Kg * A * B)
        got = gpu_fc(-a, w, False, ab, wb, np.float32(1), np.float32(1), np.float32(1))
        assert np.all(got["acc"] == -Kg * A * B)
    # largest reduction that still fits int32 at 8x8 bits
    Kg = 33025
    a = np.full((3, Kg), 1e9, np.float32)
    got = gpu_fc(a, a[:2], False, 8, 8, np.float32(1), np.float32(1), np.float32(1))
    assert np.all(got["acc"] == Kg * 255 * 255)
    # and fully anti-correlated operands at that length: S = Kg*A*B, so 2*S exceeds 2^31 inside the combine
    a = np.full((40, Kg), 1e9, np.float32)
    w = np.full((50, Kg), -1e9, np.float32)
    for lhs, rhs in ((a, w), (-a, -w)):
        got = gpu_fc(lhs, rhs, False, 8, 8, np.float32(1), np.float32(1), np.float32(1))
        assert np.all(got["acc"] == -Kg * 255 * 255)
        assert np.all(got["out"] == np.float32(-Kg * 255 * 255))


def test_bgemm_k_major_weights_relu_and_strided_output():
    import torch
    from paper_2106_09886_b200 import qnn
    rng = np.random.default_rng(12)
    a = rng.standard_normal((90, 300)).astype(np.float32)
    w = (0.05 * rng.standard_normal((300, 70))).astype(np.float32)       # [Kg][Ng]
    run_case(a, w, True, 2, 3, relu=True)
    # out only / acc only / padded leading dimension
    sa, sw, alpha = scales_for(a, w, 2, 2)
    _, _, acc, out = oracle_fc(a, w, True, 2, 2, sa, sw, alpha)
    dev = torch.device("cuda:0")
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev), 2, sa)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), 70, 1, 300, qnn.W_TCN, 2, sw)
    wide = torch.full((90, 96), 123.0, dtype=torch.float32, device=dev)
    qnn.bgemm(planes, 2, packed, 2, 90, 70, 300, alpha, out=wide[:, :70])
    assert_fp32_close(wide[:, :70].cpu().numpy(), out)
    assert torch.all(wide[:, 70:] == 123.0)
    acc_d = torch.empty((90, 70), dtype=torch.int32, device=dev)
    assert qnn.lib.qnn_bgemm(planes.data_ptr(), 2, packed.data_ptr(), 2, 90, 70, 300, float(alpha), None, 70,
                             acc_d.data_ptr(), None) == 0
    torch.cuda.synchronize()
    assert np.array_equal(acc_d.cpu().numpy(), acc)


def test_bgemm_is_deterministic():
    rng = np.random.default_rng(3)
    a = rng.standard_normal((300, 2048)).astype(np.float32)
    w = rng.standard_normal((200, 2048)).astype(np.float32)
    r1 = gpu_fc(a, w, False, 3, 3, np.float32(0.3), np.float32(0.3), np.float32(0.09))
    r2 = gpu_fc(a, w, False, 3, 3, np.float32(0.3), np.float32(0.3), np.float32(0.09))
    assert np.array_equal(r1["acc"], r2["acc"]) and np.array_equal(r1["out"].view(np.uint32), r2["out"].view(np.uint32))


def test_config1_fc_layer():
    c = wl.fc_config1(0)
    got = run_case(c.a, c.w, c.k_major, c.ab, c.wb)
    assert got["out"].shape == (64, 256)


@pytest.mark.parametrize("wb,ab", wl.GEMM_SWEEP_BITS)
def test_config3_gemm_4096_full(wb, ab):
    """Full-size square GEMM, every width pair of the sweep: all 16.7 M accumulators and outputs are compared with
    the oracle's naive integer product (about a second and a half of host time per pair)."""
    c = wl.gemm_config3(0, 4096, wb, ab)
    sa, sw, alpha = scales_for(c.a, c.w, ab, wb)
    qa, qw = oracle_fc_codes(c.a, c.w, False, ab, wb, sa, sw)
    got = gpu_fc(c.a, c.w, False, ab, wb, sa, sw, alpha, want_planes=True)
    assert np.array_equal(got["a_planes"], oracle.pack_planes(qa, ab))
    assert np.array_equal(got["w_planes"], oracle.pack_planes(qw, wb))
    want = oracle.fc(qa, qw)
    assert np.array_equal(got["acc"], want)
    assert_fp32_close(got["out"], oracle.scale(want, alpha))


def test_fc_forward_host_matches_oracle():
    """qnn_fc_forward_host: pinned host buffers in and out, device staging buffers supplied by the caller."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(21)
    a = np.abs(rng.standard_normal((300, 1000))).astype(np.float32)
    w = (0.02 * rng.standard_normal((200, 1000))).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, 2, 2)
    _, _, acc, out = oracle_fc(a, w, False, 2, 2, sa, sw, alpha)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), 200, 1, 1000, qnn.W_NTC, 2, sw)
    x_host = torch.from_numpy(a).pin_memory()
    out_host = torch.zeros((300, 200), dtype=torch.float32).pin_memory()
    x_dev = torch.empty((300, 1000), dtype=torch.float32, device=dev)
    planes = torch.empty((300, 2, qnn.row_words(1000)), dtype=torch.int32, device=dev)
    out_dev = torch.empty((300, 200), dtype=torch.float32, device=dev)
    qnn.fc_forward_host(x_host, 2, sa, 0, packed, 2, 200, alpha, out_host, x_dev, planes, out_dev)
    torch.cuda.synchronize()
    assert_fp32_close(out_host.numpy(), out)


def test_fc_forward_host_pipelined_matches_oracle():
    """Row chunks spread over three streams (ragged last chunk) give the same result as the oracle."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(22)
    a = np.abs(rng.standard_normal((1000, 700))).astype(np.float32)
    w = (0.02 * rng.standard_normal((130, 700))).astype(np.float32)
    sa, sw, alpha = scales_for(a, w, 3, 2)
    _, _, acc, out = oracle_fc(a, w, False, 3, 2, sa, sw, alpha)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), 130, 1, 700, qnn.W_NTC, 2, sw)
    x_host = torch.from_numpy(a).pin_memory()
    out_host = torch.zeros((1000, 130), dtype=torch.float32).pin_memory()
    x_dev = torch.empty((1000, 700), dtype=torch.float32, device=dev)
    planes = torch.empty((1000, 3, qnn.row_words(700)), dtype=torch.int32, device=dev)
    out_dev = torch.empty((1000, 130), dtype=torch.float32, device=dev)
    streams = [torch.cuda.Stream() for _ in range(3)]
    qnn.fc_forward_host_pipelined(x_host, 3, sa, 0, packed, 2, 130, alpha, out_host, x_dev, planes, out_dev, 192, streams)
    torch.cuda.synchronize()
    assert_fp32_close(out_host.numpy(), out)


def test_bgemm_output_beyond_2g_elements():
    """More than 2^31 outputs (8.8 GB of fp32): exercises the 64-bit output indexing.  The oracle evaluates sampled
    entries, among them the very last rows."""
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    if torch.cuda.get_device_properties(dev).total_memory < 40 * 2 ** 30:
        pytest.skip("needs about 10 GB of device memory")
    Mg, Ng, Kg, ab, wb = 2_200_000, 1000, 32, 2, 2
    assert Mg * Ng > 2 ** 31
    rng = np.random.default_rng(31)
    a = rng.standard_normal((Mg, Kg), dtype=np.float32)
    w = rng.standard_normal((Ng, Kg), dtype=np.float32)
    sa, sw, alpha = scales_for(a, w, ab, wb)
    qa, qw = oracle_fc_codes(a, w, False, ab, wb, sa, sw)
    planes = qnn.encode_pack(torch.from_numpy(a).to(dev), ab, sa)
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Ng, 1, Kg, qnn.W_NTC, wb, sw)
    out = qnn.bgemm(planes, ab, packed, wb, Mg, Ng, Kg, alpha)
    rows = np.concatenate([rng.integers(0, Mg, size=200000), np.full(1000, Mg - 1), np.full(1000, 2 ** 31 // Ng + 1)])
    cols = np.concatenate([rng.integers(0, Ng, size=200000), np.arange(1000), np.arange(1000)])
    idx = torch.from_numpy(rows.astype(np.int64) * Ng + cols.astype(np.int64)).to(dev)
    got = out.view(-1)[idx].cpu().numpy()
    del out
    want = oracle.scale(oracle.fc_sampled(qa, qw, rows, cols), alpha)
    assert_fp32_close(got, want)

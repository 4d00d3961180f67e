"""The int8 tensor-core comparison path must give the oracle's integers: bit-exact int32 accumulators and fp32
outputs (one int->float conversion and one multiply on both sides), on ragged shapes and at the benchmarked size."""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu


def _codes(rng, rows, k, bits):
    return (2 * rng.integers(0, 2 ** bits, size=(rows, k)) - (2 ** bits - 1)).astype(np.int16)


def _dev_planes(q, bits, dev):
    import torch
    return torch.from_numpy(oracle.pack_planes(q, bits).view(np.int32)).to(dev)


@pytest.mark.parametrize("Mg,Ng,Kg", [(1, 1, 1), (128, 256, 128), (130, 70, 100), (257, 300, 129), (64, 520, 1000),
                                      (300, 129, 4100)])
@pytest.mark.parametrize("ab,wb", [(1, 1), (2, 2), (3, 5), (7, 7)])
def test_int8_tensor_matches_oracle(Mg, Ng, Kg, ab, wb):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(Mg + 3 * Ng + 7 * Kg + ab)
    qa, qw = _codes(rng, Mg, Kg, ab), _codes(rng, Ng, Kg, wb)
    alpha = float(np.float32(0.013))
    want_acc = oracle.fc(qa, qw)
    out, acc = qnn.bgemm_int8_tensor(_dev_planes(qa, ab, dev), ab, _dev_planes(qw, wb, dev), wb, Mg, Ng, Kg, alpha)
    assert qnn.tensor_path_status() == 0
    assert np.array_equal(acc.cpu().numpy(), want_acc)
    assert np.array_equal(out.cpu().numpy(), oracle.scale(want_acc, alpha))


def test_int8_tensor_identical_to_bgemm_at_benchmark_size():
    import torch
    from paper_2106_09886_b200 import qnn, workloads as wl
    from helpers import scales_for
    dev = torch.device("cuda:0")
    c = wl.gemm_config3(0, 4096, 2, 2)
    sa, sw, alpha = scales_for(c.a, c.w, c.ab, c.wb)
    Mg, Kg = c.a.shape
    Ng = c.w.shape[1] if c.k_major else c.w.shape[0]
    planes = qnn.encode_pack(torch.from_numpy(c.a).to(dev), c.ab, sa)
    packed = qnn.pack_weights(torch.from_numpy(np.ascontiguousarray(c.w)).to(dev), Ng, 1, Kg,
                              qnn.W_TCN if c.k_major else qnn.W_NTC, c.wb, sw)
    out, acc = qnn.bgemm(planes, c.ab, packed, c.wb, Mg, Ng, Kg, alpha, want_acc=True)
    out8, acc8 = qnn.bgemm_int8_tensor(planes, c.ab, packed, c.wb, Mg, Ng, Kg, alpha)
    assert qnn.tensor_path_status() == 0
    assert torch.equal(acc, acc8) and torch.equal(out, out8)
    rows, cols = wl.sample_pairs(1, Mg, Ng, 200)
    qa, qw = oracle.quantize(c.a, c.ab, sa), oracle.quantize(np.ascontiguousarray(c.w.T if c.k_major else c.w), c.wb, sw)
    assert np.array_equal(acc8.cpu().numpy()[rows, cols], oracle.fc_sampled(qa, qw, rows, cols))


def test_int8_tensor_refuses_8_bit_codes():
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    planes = torch.zeros((8, 8, 4), dtype=torch.int32, device=dev)
    with pytest.raises(qnn.QnnError) as e:
        qnn.bgemm_int8_tensor(planes, 8, planes, 2, 8, 8, 8, 1.0)
    assert "range" in str(e.value)

"""The give-up path of the tensor-path kernels' bounded waits, made to run on purpose without faulting anything.

qnn_selftest_bounded_wait launches one small block, built from the same wait helpers as the tcgen05 GEMM kernel, in
which a producer waits for a stage release that nobody gives.  The wait runs out after the given number of polls, the
block raises its abort flag and the library's status word, drains its copy in flight and ends normally.  Checked
here: the status call reports QNN_E_DEVICE with the id of that wait, reading clears the record, and an ordinary
backward product right afterwards is still exact (the context and the library are unaffected).
"""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu


def _exact_backward_product(qnn, torch, seed):
    rng = np.random.default_rng(seed)
    m, n, k, wb = 200, 136, 300, 3
    qw = (2 * rng.integers(0, 2 ** wb, size=(n, k)) - (2 ** wb - 1)).astype(np.int16)
    g = rng.integers(-8, 9, size=(m, n)).astype(np.float32)
    dev = torch.device("cuda:0")
    planes = torch.from_numpy(oracle.pack_planes(qw, wb).view(np.int32)).to(dev)
    G = qnn.bgemm_backward_data(torch.from_numpy(g).to(dev), planes, k, wb, 0.5).cpu().numpy()
    want = oracle.fc_backward_data(g, qw, 1, wb, 0.5)[0]
    assert np.array_equal(G.astype(np.float64), want)


@pytest.mark.parametrize("limit", [64, 1024, 5000])
def test_a_wait_that_runs_out_is_reported_and_leaves_the_library_usable(limit):
    import torch
    from paper_2106_09886_b200 import qnn
    rc, word = qnn.last_device_status()
    assert (rc, word) == (qnn.OK, 0)                       # nothing pending from earlier tests
    _exact_backward_product(qnn, torch, 1)
    assert qnn.tensor_path_status() == 0                   # the real kernels' waits all ended by an arrival
    qnn.selftest_bounded_wait(limit)
    rc, word = qnn.last_device_status()
    assert rc == qnn.E_DEVICE and word == 1                # 1 + wait id 0: the producer's wait for a free stage
    assert "internal error" in qnn.status_string(rc)
    assert qnn.last_device_status() == (qnn.OK, 0)         # reading cleared the record
    with pytest.raises(qnn.QnnError):                      # the raising form of the same call
        qnn.selftest_bounded_wait(limit)
        qnn.tensor_path_status()
    _exact_backward_product(qnn, torch, 2)
    assert qnn.tensor_path_status() == 0


def test_selftest_rejects_limits_outside_its_range():
    from paper_2106_09886_b200 import qnn
    assert qnn.lib.qnn_selftest_bounded_wait(0, None) == qnn.E_ARG
    assert qnn.lib.qnn_selftest_bounded_wait(1 << 20, None) == qnn.E_ARG
    assert qnn.lib.qnn_last_device_status(None) == qnn.E_ARG

"""qnn_fc_forward_noalloc: the FC layer for callers that cannot allocate device memory.

Such a caller (a framework plug-in that must not allocate in its callback, a real-time loop with memory
fixed at start-up, a bare C program) passes only its input, the packed weights and its output; the
activation planes in between live in an array built into the library.  The check: through the C ABI, its
output equals that of the ordinary two-call route (qnn_encode_pack into a caller-allocated buffer, then
qnn_bgemm) and the CPU oracle's result for the same layer, on two calls in a row that share the built-in
array -- the second with a different, smaller problem, so that planes left over from the first call would
show up if they leaked.

This file sorts last on purpose: a run that stops at the first failure has then already run every other test.
"""
import ctypes

import numpy as np
import pytest

from helpers import assert_fp32_close, oracle_fc

pytestmark = pytest.mark.gpu


def _two_call_route(qnn, torch, x_d, packed, ab, wb, sa, alpha, Ng, flags):
    Mg, Kg = x_d.shape
    planes = qnn.encode_pack(x_d, ab, sa, flags)
    out = qnn.bgemm(planes, ab, packed, wb, Mg, Ng, Kg, alpha)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def test_noalloc_entry_matches_two_call_route_twice_in_a_row():
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(77)
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    cases = [(700, 300, 1500, 3, 2, qnn.RELU), (64, 256, 512, 2, 2, 0)]       # (Mg, Ng, Kg, ab, wb, flags)
    for Mg, Ng, Kg, ab, wb, flags in cases:
        x = rng.standard_normal((Mg, Kg)).astype(np.float32)
        w = (0.05 * rng.standard_normal((Ng, Kg))).astype(np.float32)
        sa = np.float32(np.abs(x).max()) / np.float32(2 ** ab - 1)
        sw = np.float32(np.abs(w).max()) / np.float32(2 ** wb - 1)
        alpha = np.float32(sa * sw)
        x_d = torch.from_numpy(x).to(dev)
        packed = qnn.pack_weights(torch.from_numpy(w).to(dev), Ng, 1, Kg, qnn.W_NTC, wb, sw)
        want = _two_call_route(qnn, torch, x_d, packed, ab, wb, sa, alpha, Ng, flags)
        out = torch.full((Mg, Ng), float("nan"), dtype=torch.float32, device=dev)
        rc = qnn.lib.qnn_fc_forward_noalloc(ctypes.c_void_p(x_d.data_ptr()), Mg, Kg, Kg, ab, float(sa), flags,
                                            ctypes.c_void_p(packed.data_ptr()), wb, Ng, float(alpha),
                                            ctypes.c_void_p(out.data_ptr()), Ng, stream)
        assert rc == qnn.OK, qnn.status_string(rc)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.all(np.abs(got.astype(np.float64) - want) <= 1e-6 * np.abs(want.astype(np.float64)))
        assert np.array_equal(got, want)                    # same kernels, same inputs: the same bits
        # and against the independent CPU oracle, so that a mistake common to both GPU routes cannot pass
        _, _, _, want_oracle = oracle_fc(x, w, False, ab, wb, sa, sw, alpha, relu=bool(flags & qnn.RELU))
        assert_fp32_close(got, want_oracle)


def test_noalloc_entry_refuses_what_does_not_fit():
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    x = torch.zeros((8, 64), dtype=torch.float32, device=dev)
    packed = qnn.pack_weights(torch.ones((8, 64), dtype=torch.float32, device=dev), 8, 1, 64, qnn.W_NTC, 2, 1.0)
    out = torch.zeros((8, 8), dtype=torch.float32, device=dev)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    # 16384 rows x 4096 elements at 2 bits need 16 MiB of planes: more than the built-in 8 MiB
    assert qnn.planes_bytes(16384, 4096, 2) > qnn.NOALLOC_SCRATCH_BYTES
    assert qnn.lib.qnn_fc_forward_noalloc(p(x), 16384, 4096, 4096, 2, 1.0, 0, p(packed), 2, 8, 1.0, p(out), 8, None) == qnn.E_RANGE
    assert qnn.lib.qnn_fc_forward_noalloc(None, 8, 64, 64, 2, 1.0, 0, p(packed), 2, 8, 1.0, p(out), 8, None) == qnn.E_ARG
    assert qnn.lib.qnn_fc_forward_noalloc(p(x), 8, 64, 64, 2, 0.0, 0, p(packed), 2, 8, 1.0, p(out), 8, None) == qnn.E_SCALE
    # the largest problem that fits exactly is accepted by the size check (4096 x 4096 at 4 bits = 8 MiB)
    assert qnn.planes_bytes(4096, 4096, 4) == qnn.NOALLOC_SCRATCH_BYTES

"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and its host-side
argument validation and size queries behave as the header says.  No kernel is launched here."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

import oracle

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def qnn():
    from paper_2106_09886_b200 import build
    build.build()
    from paper_2106_09886_b200 import qnn as q
    return q


def declared_functions():
    text = (ROOT / "include" / "qnn.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qnn_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(qnn):
    names = declared_functions()
    assert "qnn_bgemm" in names and "qnn_bconv2d" in names and "qnn_encode_pack" in names and "qnn_pack_weights" in names
    for name in names:
        assert hasattr(qnn.lib, name), name
    assert sorted(qnn.EXPORTS) == names


def test_size_queries_match_layout(qnn):
    for k in [1, 31, 32, 33, 127, 128, 129, 512, 4096, 4097]:
        assert qnn.row_words(k) == oracle.row_words(k)
        assert qnn.planes_bytes(7, k, 3) == 7 * 3 * oracle.row_words(k) * 4
    assert qnn.row_words(0) == 0 and qnn.planes_bytes(0, 5, 2) == 0 and qnn.planes_bytes(5, 5, 9) == 0
    # conv weights: every tap starts on a word boundary
    assert qnn.weights_row_words(9, 256) == 72 and qnn.weights_row_words(9, 3) == 12 and qnn.weights_row_words(1, 64) == 4
    assert qnn.weights_bytes(256, 9, 256, 2) == 256 * 2 * 72 * 4 + 256 * 9 * 4
    assert qnn.weights_bytes(5, 1, 40, 3) == 5 * 3 * 4 * 4 + 32       # tapsum rounded up to 16 bytes
    # Table 3's compression column: 32/bits
    for bits in range(1, 9):
        assert qnn.planes_bytes(64, 4096, bits) * bits == 64 * 4096 * 4 * bits * bits // 32


def test_status_strings_and_version(qnn):
    assert qnn.version() >= 100
    seen = {qnn.status_string(s) for s in range(0, -7, -1)}
    assert len(seen) == 7 and qnn.status_string(0) == "ok" and qnn.status_string(-99) == "unknown status"


def test_argument_errors_are_reported_before_any_launch(qnn):
    lib = qnn.lib
    buf = (ctypes.c_char * 4096)()
    base = ctypes.addressof(buf)
    p = ctypes.c_void_p((base + 15) // 16 * 16)                    # aligned, never dereferenced by these calls
    mis = ctypes.c_void_p(p.value + 4)
    assert lib.qnn_encode_pack(None, 4, 64, 64, 2, 1.0, 0, p, None, None) == qnn.E_ARG
    assert lib.qnn_encode_pack(p, 4, 64, 32, 2, 1.0, 0, p, None, None) == qnn.E_ARG       # ldx < k
    assert lib.qnn_encode_pack(p, 4, 64, 64, 9, 1.0, 0, p, None, None) == qnn.E_ARG
    assert lib.qnn_encode_pack(p, 4, 64, 64, 2, 1.0, 2, p, None, None) == qnn.E_ARG       # unknown flag
    assert lib.qnn_encode_pack(p, 4, 64, 64, 2, 0.0, 0, p, None, None) == qnn.E_SCALE
    assert lib.qnn_encode_pack(p, 4, 64, 64, 2, float("nan"), 0, p, None, None) == qnn.E_SCALE
    assert lib.qnn_encode_pack(p, 4, 64, 64, 2, 1.0, 0, mis, None, None) == qnn.E_ALIGN
    assert lib.qnn_pack_weights(p, 4, 1, 64, 7, 2, 1.0, p, None) == qnn.E_ARG            # unknown layout
    assert lib.qnn_pack_weights(p, 4, 1, 64, 0, 2, -1.0, p, None) == qnn.E_SCALE
    assert lib.qnn_pack_weights(p, 4, 1, 64, 0, 2, 1.0, mis, None) == qnn.E_ALIGN
    assert lib.qnn_bgemm(p, 2, p, 2, 4, 4, 64, 1.0, None, 4, None, None) == qnn.E_ARG    # no output at all
    assert lib.qnn_bgemm(p, 0, p, 2, 4, 4, 64, 1.0, p, 4, None, None) == qnn.E_ARG
    assert lib.qnn_bgemm(p, 2, p, 2, 4, 4, 64, 1.0, p, 3, None, None) == qnn.E_ARG       # ldo < Ng
    assert lib.qnn_bgemm(p, 2, p, 2, 4, 4, 64, float("inf"), p, 4, None, None) == qnn.E_SCALE
    assert lib.qnn_bgemm(mis, 2, p, 2, 4, 4, 64, 1.0, p, 4, None, None) == qnn.E_ALIGN
    assert lib.qnn_bgemm(p, 8, p, 8, 4, 4, 33026, 1.0, p, 4, None, None) == qnn.E_RANGE  # 33026*255*255 >= 2^31
    assert lib.qnn_bconv2d(p, 2, p, 2, 1, 4, 4, 8, 8, 3, 3, 0, 1, 1.0, p, None, None) == qnn.E_ARG   # stride 0
    assert lib.qnn_bconv2d(p, 2, p, 2, 1, 2, 2, 8, 8, 5, 5, 1, 0, 1.0, p, None, None) == qnn.E_ARG   # kernel > image
    assert lib.qnn_bconv2d(p, 8, p, 8, 1, 8, 8, 4096, 8, 3, 3, 1, 1, 1.0, p, None, None) == qnn.E_RANGE
    # empty problems are refused, not launched
    assert lib.qnn_encode_pack(p, 0, 64, 64, 2, 1.0, 0, p, None, None) == qnn.E_ARG
    assert lib.qnn_encode_pack(p, 4, 0, 0, 2, 1.0, 0, p, None, None) == qnn.E_ARG
    assert lib.qnn_pack_weights(p, 0, 1, 64, 0, 2, 1.0, p, None) == qnn.E_ARG
    assert lib.qnn_bgemm(p, 2, p, 2, 0, 4, 64, 1.0, p, 4, None, None) == qnn.E_ARG
    assert lib.qnn_bgemm(p, 2, p, 2, 4, 0, 64, 1.0, p, 4, None, None) == qnn.E_ARG
    assert lib.qnn_bgemm(p, 2, p, 2, 4, 4, 0, 1.0, p, 4, None, None) == qnn.E_ARG
    assert lib.qnn_bconv2d(p, 2, p, 2, 0, 4, 4, 8, 8, 3, 3, 1, 1, 1.0, p, None, None) == qnn.E_ARG
    assert lib.qnn_absmax_f32(p, 0, p, None) == qnn.E_ARG
    assert lib.qnn_absmax_f32(None, 4, p, None) == qnn.E_ARG
    assert lib.qnn_probe_copy(p, p, 24, None) == qnn.E_ARG
    assert lib.qnn_probe_naive_sgemm(p, p, None, 4, 4, 4, None) == qnn.E_ARG
    assert lib.qnn_probe_naive_sgemm(p, p, p, 4, 0, 4, None) == qnn.E_ARG
    assert lib.qnn_probe_naive_sgemm(p, p, p, 8 * 65535 + 1, 4, 4, None) == qnn.E_RANGE


def test_composite_calls_check_every_argument_before_their_first_copy_or_launch(qnn):
    """qnn_fc_forward_host, its pipelined form and qnn_fc_forward_noalloc wrap a copy, the encoder and the contraction:
    an argument that only the contraction would refuse (weight width, alpha, the int32 range, a misaligned blob)
    must come back as an error with nothing enqueued.  On a machine without a GPU a copy or launch would answer
    QNN_E_CUDA instead, so the exact codes below also show that nothing was attempted."""
    lib = qnn.lib
    buf = (ctypes.c_char * 4096)()
    p = ctypes.c_void_p((ctypes.addressof(buf) + 255) // 256 * 256)      # aligned, never dereferenced by these calls
    mis = ctypes.c_void_p(p.value + 4)
    streams = (ctypes.c_void_p * 2)(None, None)
    inf, nan = float("inf"), float("nan")

    def host(wb=2, alpha=1.0, Kg=64, w=p, ab=2, scale=1.0, flags=0):
        return lib.qnn_fc_forward_host(p, 4, Kg, ab, scale, flags, w, wb, 4, alpha, p, p, p, p, None)

    def piped(wb=2, alpha=1.0, Kg=64, w=p, ab=2, scale=1.0, flags=0):
        return lib.qnn_fc_forward_host_pipelined(p, 4, Kg, ab, scale, flags, w, wb, 4, alpha, p, p, p, p, 2, streams, 2)

    def noalloc(wb=2, alpha=1.0, Kg=64, w=p, ab=2, scale=1.0, flags=0):
        return lib.qnn_fc_forward_noalloc(p, 4, Kg, Kg, ab, scale, flags, w, wb, 4, alpha, p, 4, None)

    for call in (host, piped, noalloc):
        assert call(wb=0) == qnn.E_ARG and call(wb=9) == qnn.E_ARG
        assert call(alpha=inf) == qnn.E_SCALE and call(alpha=nan) == qnn.E_SCALE
        assert call(ab=8, wb=8, Kg=33026) == qnn.E_RANGE                  # 33026*255*255 >= 2^31
        assert call(w=mis) == qnn.E_ALIGN
        assert call(scale=0.0) == qnn.E_SCALE and call(flags=2) == qnn.E_ARG and call(ab=9) == qnn.E_ARG


def test_popcounts_per_output_mirror_the_dispatch(qnn):
    """The roofline helper: popcount instructions per output element of the kernel that serves a layer."""
    f = qnn.lib.qnn_popcounts_per_output
    # fully-connected, Kg = 4096: 128 words = 16 groups of 8 words at 4 popcounts, for each of the ab*wb pairs
    assert f(2, 2, 0, 1, 1, 4096, 4096) == 4 * 16 * 4 and f(1, 1, 0, 1, 1, 4096, 4096) == 16 * 4
    assert f(2, 2, 0, 1, 1, 512, 256) == 4 * 2 * 4                       # the small FC layer: 16 words
    # 3x3 convolutions: 9-word groups (4 popcounts per channel word) up to 128 channels, 8-word groups beyond
    assert f(3, 3, 1, 3, 3, 64, 64) == 9 * 2 * 4 and f(4, 4, 1, 3, 3, 128, 128) == 16 * 4 * 4
    assert f(2, 2, 1, 3, 3, 256, 256) == 4 * 9 * 4                       # 72 words = 9 groups of 8
    assert f(5, 3, 1, 3, 3, 64, 64) == 15 * (2 * 4 + 2)                  # 18 words: two groups and a tail of two words
    # short reductions: the adder tree across plane pairs stops at W/2 adders (W = ab*wb*words)
    assert f(3, 3, 1, 1, 1, 64, 128) == 9 and f(3, 3, 1, 1, 1, 128, 256) == 18 and f(4, 4, 0, 1, 1, 128, 64) == 32
    assert f(1, 1, 0, 1, 1, 32, 8) == 1
    # whole patch in one word (first layer on 3 channels): 10 popcounts at 4 x 4 bits, 7 at 3 x 3, one per pair otherwise
    assert f(4, 4, 1, 3, 3, 3, 64) == 10 and f(3, 3, 1, 3, 3, 3, 64) == 7 and f(2, 4, 1, 3, 3, 3, 64) == 8
    assert f(0, 2, 0, 1, 1, 64, 8) == 0 and f(2, 2, 0, 3, 3, 64, 8) == 0 and f(2, 9, 1, 3, 3, 64, 8) == 0


def test_status_calls_check_their_arguments_on_the_host(qnn):
    assert qnn.lib.qnn_selftest_bounded_wait(0, None) == qnn.E_ARG
    assert qnn.lib.qnn_selftest_bounded_wait(1 << 20, None) == qnn.E_ARG
    assert qnn.lib.qnn_last_device_status(None) == qnn.E_ARG and qnn.lib.qnn_tensor_path_status(None) == qnn.E_ARG


def test_importing_binding_without_library_fails_loudly(tmp_path, monkeypatch):
    import importlib.util
    src = (ROOT / "paper_2106_09886_b200" / "qnn.py").read_text()
    mod_path = tmp_path / "qnn_copy.py"
    mod_path.write_text(src)
    spec = importlib.util.spec_from_file_location("qnn_copy", mod_path)
    with pytest.raises(ImportError):
        spec.loader.exec_module(importlib.util.module_from_spec(spec))


def test_workloads_are_seeded_and_shaped():
    from paper_2106_09886_b200 import workloads as wl
    c1, c1b = wl.fc_config1(0), wl.fc_config1(0)
    assert np.array_equal(c1.a, c1b.a) and c1.a.shape == (64, 512) and c1.w.shape == (512, 256) and c1.k_major
    assert c1.a.min() >= 0 and c1.a.max() <= 3.0 and (c1.Mg, c1.Ng, c1.Kg) == (64, 256, 512)
    c2 = wl.conv_config2(0, batch=2)
    assert c2.a.shape == (2, 14, 14, 256) and c2.w.shape == (256, 3, 3, 256) and c2.a.min() >= 0
    assert wl.conv_config2(0).shape.Mg == 6272 and wl.conv_config2(0).shape.Kg == 2304
    r = wl.resnet18_shapes()
    assert len(r) == 19 and sum(s.int_macs for s in r) // 10 ** 9 == 434
    v = wl.vgg16_shapes()
    assert len(v) == 13 and sum(s.int_macs for s in v) // 10 ** 9 == 982
    assert v[0].Kg == 27 and v[0].Mg == 3211264


def test_mixed_precision_resnet18_reproduces_table4_compression():
    """Table 4: per-stage widths of Precision#1 / #2 give 5.0x / 14.1x weight compression with one bit per
    element per plane; the packed blobs of the quantized convolutions hold those plane bits, each (feature, plane)
    row rounded up to 16 bytes, plus the per-tap sums."""
    from paper_2106_09886_b200 import workloads as wl
    for precision, want in ((1, 5.0), (2, 14.1)):
        q, full = wl.resnet18_weight_bits(precision)
        assert abs(full / q - want) < 0.06, (precision, full / q)
        assert wl.RESNET18_MIXED[precision]["compression"] == want
    from paper_2106_09886_b200 import build
    build.build()
    from paper_2106_09886_b200 import qnn
    tot_ideal = tot_rows = 0
    for s in wl.resnet18_mixed_shapes(2, batch=1):
        ideal = s.Cout * s.R * s.S * s.C * s.wb // 8
        row = (s.R * s.S * s.C // 32 + 3) // 4 * 4 * 4                     # bytes of one (feature, plane) row
        got = qnn.weights_bytes(s.Cout, s.R * s.S, s.C, s.wb)
        assert got == s.Cout * s.wb * row + (s.Cout * s.R * s.S * 4 + 15) // 16 * 16
        tot_ideal += ideal
        tot_rows += s.Cout * s.wb * row
    assert tot_ideal <= tot_rows <= 1.01 * tot_ideal      # row padding costs under 1% over the whole network
